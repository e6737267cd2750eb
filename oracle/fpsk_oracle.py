"""FP64 CPU oracle of the FP-Sketch verifier (test infrastructure, not product).

Everything here is written straight from the paper's definitions: the error
matrix E = AB - C is formed explicitly in FP64 and every sketch is a plain sum
over E.  Nothing is blocked, fused or reordered.  numpy's matmul, sort and
bincount serve as library steps.  The module imports nothing from the CUDA
package and the CUDA package imports nothing from here.

Notation follows the paper: A is n1 x n2, B is n2 x n3, C is n1 x n3 (FP32),
m is the bucket count per side (written ``m_b`` in code), hashes h1, h2 and
signs v1, v2, sketches S, R, T, radius r, confirmed set F.

Indices are 0-based in every interface; the 1-based index weights
w_i = (i+1)/2^ceil(log2 n1) are internal.

Parity pins (tests/test_oracle_*.py): integer brute force for Eq. (S),
exact single-fault recovery for Eq. (recover), peeling against the term-by-term
sketch of the faults left behind (exact on integer products), the printed bucket
counts of Table "rect" and the other integers the paper prints for the sizing law,
Gaussian closed forms for the two noise estimators and for the normalisation of
the noise constant, brute force for the tolerance denominators, collision
statistics for the hash rounds, Lemma 1 on a clean product.  Two readings have no
pin in the paper and are "parity unpinned": the probe threshold applied to the
un-hashed column sketch (bucket count taken as n3, analytic cap scaled by
sqrt(n1)), and the value of the noise constant on a given GPU (the paper states
that it belongs to the BLAS).  The hashed S only probe follows the rule of
Section "Thresholds" as printed.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import List, Optional, Tuple

import numpy as np

__all__ = [
    "FP16", "BF16", "EPS32", "Params", "Fault", "ProbeResult", "NoiseResult",
    "mix32", "round_key", "hash_round",
    "error_matrix", "abs_product",
    "probe_sketch", "probe_sketch_from_operands", "probe_verdict", "analytic_tau",
    "index_weights", "moment_sketches", "moment_sketches_compressed", "abs_sketch",
    "peel", "lower_median", "sigma_clip", "sigma_mad",
    "select_candidates", "decode_candidates", "search_offsets", "validate_entry",
    "localize_round", "localize",
    "c_f", "law_sigma", "m_comb", "m_max", "m_mem", "m_num", "m_start", "cap_K",
    "rms_c_estimate", "index_budget", "radius_from_budget", "plan", "recalibrated_m",
    "measure_noise", "scan_out_of_range", "apply_corrections", "verify_repair", "FP32_MAX",
    "hashed_sum_sketch", "probe_hashed", "ProbeState", "recalibration_due", "recalibrate_probe",
]

EPS32 = 2.0 ** -23          # FP32 machine epsilon used by the thresholds (Section "Validation")
GOLDEN = 0x9E3779B9
FP16, BF16 = 0, 1


# ----------------------------------------------------------------------------
# parameters and records
# ----------------------------------------------------------------------------
@dataclass
class Params:
    """Defaults of Section "Methodology" (k=3, rho_min=0.02, r*=4, r_max=16),
    Section "Validation" (c=100), Section "Thresholds" (mu=4, k_MAD=2) and
    Section "Sketch Noise Sets the Bucket Count" (B*=0.3, collision c=2).
    s_budget and delta_max are the declared fault count s and the per-line
    bound Delta; 8 and 8 reproduce the floor of 48 seen in Table "rect"."""
    rounds: int = 3
    rho_min: float = 0.02
    r_star: int = 4
    r_max: int = 16
    radius: int = -1            # -1: take the radius from the calibration plan
    c_valid: float = 100.0
    mu: float = 4.0
    b_star: float = 0.3
    c_coll: float = 2.0
    s_budget: int = 8
    delta_max: int = 8
    mad_of_abs: int = 1         # 1: MAD of |S| as printed; 0: signed MAD of S
    scale_cap: int = 0          # hashed probe only. 0: thr = min(tau, ...) as printed in Section
                                # "Thresholds"; 1: the cap enters as tau sqrt(n1 n3 / m^2)


@dataclass
class Fault:
    i: int
    j: int
    delta: float                # gamma - C_ij  (the correction of Section "Validation")
    recompute: float            # gamma
    c_value: float
    round: int
    bucket_a: int
    bucket_b: int


@dataclass
class ProbeResult:
    fired: bool
    nonfinite: bool
    argmax_col: int
    max_abs: float
    sigma_hat: float
    thr: float
    tau: float


@dataclass
class NoiseResult:
    sigma_clip: float
    sigma_mad: float
    rms_c: float
    c_hat: float
    index_budget_B: float
    m0: int
    m_probe: int
    m_loc: int
    radius: int


# ----------------------------------------------------------------------------
# hash rounds  (Section "Moment Sketches": "draw hashes h1, h2 and signs v1, v2";
# the paper fixes no family, this integer hash is this build's written reading)
# ----------------------------------------------------------------------------
def mix32(x):
    """Two multiply/xor-shift rounds on 32-bit words (numpy uint64 carrier)."""
    x = np.asarray(x, dtype=np.uint64) & np.uint64(0xFFFFFFFF)
    x = x ^ (x >> np.uint64(16))
    x = (x * np.uint64(0x7FEB352D)) & np.uint64(0xFFFFFFFF)
    x = x ^ (x >> np.uint64(15))
    x = (x * np.uint64(0x846CA68B)) & np.uint64(0xFFFFFFFF)
    x = x ^ (x >> np.uint64(16))
    return x


def round_key(seed: int, rnd: int, side: int) -> int:
    """32-bit key of (seed, hash round, side); side 0 = rows (h1,v1), 1 = columns (h2,v2)."""
    lo = seed & 0xFFFFFFFF
    hi = (seed >> 32) & 0xFFFFFFFF
    inner = int(mix32((hi + GOLDEN * (2 * rnd + side + 1)) & 0xFFFFFFFF))
    return int(mix32(lo ^ inner))


def hash_round(seed: int, rnd: int, side: int, n: int, m_b: int) -> Tuple[np.ndarray, np.ndarray]:
    """Bucket h(idx) in [0, m_b) and sign v(idx) in {+1,-1} for idx = 0..n-1."""
    key = np.uint64(round_key(seed, rnd, side))
    idx = np.arange(n, dtype=np.uint64)
    h = mix32(idx ^ key)
    bucket = ((h * np.uint64(m_b)) >> np.uint64(32)).astype(np.int64)
    sbit = mix32((h + np.uint64(GOLDEN)) & np.uint64(0xFFFFFFFF)) & np.uint64(1)
    sign = np.where(sbit == 0, 1.0, -1.0)
    return bucket, sign


# ----------------------------------------------------------------------------
# the error matrix and the probe  (Introduction: E = AB - C;  Eq. (S) with
# H1 = 1^T and H2 = I gives the column-sum sketch s = 1^T E)
# ----------------------------------------------------------------------------
def _f64(x):
    return np.ascontiguousarray(np.asarray(x, dtype=np.float64))


def error_matrix(A, B, C) -> np.ndarray:
    """E = AB - C in FP64 (products of two half-precision values are exact in FP64)."""
    return _f64(A) @ _f64(B) - _f64(C)


def abs_product(A, B) -> np.ndarray:
    """sum_k |A_ik||B_kj|: the denominator of the parity tolerance and of tau_ij."""
    return np.abs(_f64(A)) @ np.abs(_f64(B))


def probe_sketch(E: np.ndarray) -> np.ndarray:
    """s_j = sum_i E_ij, straight from the definition."""
    return np.asarray(E, dtype=np.float64).sum(axis=0)


def probe_sketch_from_operands(A, B, C) -> np.ndarray:
    """The same sketch without forming AB: (1^T A) B - 1^T C  (Eq. (S))."""
    u = _f64(A).sum(axis=0)
    return u @ _f64(B) - _f64(C).sum(axis=0)


def analytic_tau(A, B, n2: int) -> float:
    """tau = 100 n2 eps max|A| max|B|  (Section "Thresholds")."""
    ma = float(np.max(np.abs(A))) if np.size(A) else 0.0
    mb = float(np.max(np.abs(B))) if np.size(B) else 0.0
    return 100.0 * n2 * EPS32 * ma * mb


def sigma_clip(S) -> float:
    """1.2533 mean(min(|S|, 5 mean|S|))  (Section "Thresholds", probe estimate)."""
    a = np.abs(np.asarray(S, dtype=np.float64)).ravel()
    if a.size == 0:
        return 0.0
    mean_abs = a.mean()
    return float(1.2533 * np.minimum(a, 5.0 * mean_abs).mean())


def probe_verdict(s: np.ndarray, tau: float, params: Params = None, n_rows: int = 1) -> ProbeResult:
    """thr = min(tau sqrt(n_rows), mu sqrt(2 ln N_b) sigma_hat); dirty iff max|s| > thr or s is
    not finite (Section "Thresholds", Algorithm 2 probe part, Section "Nonfinite").
    N_b is the number of sketch entries: n3 here, m^2 in the paper's hashed probe.
    n_rows is the number of entries of E that one sketch entry sums (n1 for the column
    sketch): the analytic cap tau bounds the rounding of ONE inner product (with slack 100),
    and a sum of n_rows of them grows like sqrt(n_rows); with n_rows = 1 this is the paper's
    rule verbatim.  (Reading for the un-hashed sketch; unpinned by the paper.)"""
    params = params or Params()
    s = np.asarray(s, dtype=np.float64)
    n_b = max(int(s.size), 2)
    nonfinite = bool(np.any(~np.isfinite(s)))
    sig = sigma_clip(s)
    thr = min(tau * math.sqrt(float(n_rows)), params.mu * math.sqrt(2.0 * math.log(n_b)) * sig)
    a = np.abs(s)
    if s.size:
        # NaN entries never win the argmax of the finite comparison
        a_cmp = np.where(np.isnan(a), -1.0, a)
        arg = int(np.argmax(a_cmp))
        mx = float(a_cmp[arg])
    else:
        arg, mx = -1, 0.0
    fired = bool(nonfinite or (mx > thr))
    return ProbeResult(fired, nonfinite, arg, mx, sig, thr, tau)


# ----------------------------------------------------------------------------
# the paper's own probe: S alone at the probe's bucket count m
# (Section "The Cheap S Only Probe", Eq. (S), Section "Thresholds")
# ----------------------------------------------------------------------------
def hashed_sum_sketch(E, h1, v1, h2, v2, m_b: int) -> np.ndarray:
    """S = H1 E H2^T, entry by entry from the definition (no R, no T)."""
    E = np.asarray(E, dtype=np.float64)
    flat = (np.asarray(h1, dtype=np.int64)[:, None] * m_b + np.asarray(h2, dtype=np.int64)[None, :]).ravel()
    sE = (np.asarray(v1)[:, None] * np.asarray(v2)[None, :]) * E
    with np.errstate(invalid="ignore"):
        return np.bincount(flat, weights=sE.ravel(), minlength=m_b * m_b).reshape(m_b, m_b)


def probe_hashed(A, B, C, seed: int, rnd: int, m_b: int, params: Params = None):
    """The S only probe: hash round (seed, rnd) with m_b buckets per side, S = H1 (AB - C) H2^T,
    sigma_hat = clipped mean over the m_b^2 buckets, thr = min(tau, mu sqrt(2 ln m_b^2) sigma_hat)
    as Section "Thresholds" prints it, dirty iff max|S| > thr or S is not finite.  Only with
    params.scale_cap = 1 (off by default, not in the paper) the cap enters as
    tau sqrt(n1 n3 / m_b^2), the root of the number of entries of E a bucket sums on average.
    Returns (ProbeResult with argmax_col = flat bucket index a*m_b + b, S)."""
    params = params or Params()
    A64, B64 = _f64(A), _f64(B)
    n1, n2 = A64.shape
    n3 = B64.shape[1]
    h1, v1 = hash_round(seed, rnd, 0, n1, m_b)
    h2, v2 = hash_round(seed, rnd, 1, n3, m_b)
    with np.errstate(invalid="ignore", over="ignore"):
        E = A64 @ B64 - np.asarray(C, dtype=np.float64)
    S = hashed_sum_sketch(E, h1, v1, h2, v2, m_b)
    tau = analytic_tau(A64, B64, n2)
    pop = float(n1) * float(n3) / (float(m_b) * float(m_b)) if params.scale_cap else 1.0
    return probe_verdict(S.ravel(), tau, params, n_rows=pop), S


# ----------------------------------------------------------------------------
# moment sketches  (Section "Moment Sketches", Eq. (S) and the definitions of R, T)
# ----------------------------------------------------------------------------
def index_weights(n: int) -> np.ndarray:
    """w_x = x / 2^ceil(log2 n) for x = 1..n."""
    p = (n - 1).bit_length() if n > 1 else 0
    return np.arange(1, n + 1, dtype=np.float64) / float(1 << p)


def moment_sketches(E, h1, v1, h2, v2, m_b: int):
    """S[a,b] = sum v1(i)v2(j) E_ij over h1(i)=a, h2(j)=b; R and T with the row
    weight w_i and the column weight w_j.  Definition, entry by entry."""
    E = np.asarray(E, dtype=np.float64)
    n1, n3 = E.shape
    wi = index_weights(n1)
    wj = index_weights(n3)
    flat = (np.asarray(h1, dtype=np.int64)[:, None] * m_b + np.asarray(h2, dtype=np.int64)[None, :]).ravel()
    sE = (np.asarray(v1)[:, None] * np.asarray(v2)[None, :]) * E
    mm = m_b * m_b
    S = np.bincount(flat, weights=sE.ravel(), minlength=mm).reshape(m_b, m_b)
    R = np.bincount(flat, weights=(wi[:, None] * sE).ravel(), minlength=mm).reshape(m_b, m_b)
    T = np.bincount(flat, weights=(sE * wj[None, :]).ravel(), minlength=mm).reshape(m_b, m_b)
    return S, R, T


def _H(h, v, m_b, n):
    H = np.zeros((m_b, n), dtype=np.float64)
    H[np.asarray(h, dtype=np.int64), np.arange(n)] = v
    return H


def moment_sketches_compressed(A, B, C, h1, v1, h2, v2, m_b: int):
    """The right-hand side of Eq. (S): (H1 A)(B H2^T) - H1 C H2^T and its weighted
    forms, with explicit H matrices.  Independent of moment_sketches()."""
    A, B, C = _f64(A), _f64(B), _f64(C)
    n1, n3 = C.shape
    H1 = _H(h1, v1, m_b, n1)
    H2 = _H(h2, v2, m_b, n3)
    W1 = np.diag(index_weights(n1))
    W2 = np.diag(index_weights(n3))
    P, Pw = H1 @ A, H1 @ W1 @ A
    Q, Qw = B @ H2.T, B @ W2 @ H2.T
    S = P @ Q - H1 @ C @ H2.T
    R = Pw @ Q - H1 @ W1 @ C @ H2.T
    T = P @ Qw - H1 @ C @ W2 @ H2.T
    return S, R, T


def abs_sketch(ABS, h1, h2, m_b: int) -> np.ndarray:
    """sum over the bucket of sum_k |A_ik||B_kj|: denominator of the 1e-5 sketch tolerance."""
    flat = (np.asarray(h1, dtype=np.int64)[:, None] * m_b + np.asarray(h2, dtype=np.int64)[None, :]).ravel()
    return np.bincount(flat, weights=np.asarray(ABS, dtype=np.float64).ravel(),
                       minlength=m_b * m_b).reshape(m_b, m_b)


def peel(S, R, T, F: List[Fault], h1, v1, h2, v2, n1: int, n3: int):
    """Subtract v1(i)v2(j) delta (1, w_i, w_j) of every confirmed fault at its bucket
    (Algorithm 1, peeling loop; Section "Peeling Across Hash Rounds")."""
    wi = index_weights(n1)
    wj = index_weights(n3)
    for f in F:
        a, b = int(h1[f.i]), int(h2[f.j])
        g = v1[f.i] * v2[f.j] * f.delta
        S[a, b] -= g
        R[a, b] -= g * wi[f.i]
        T[a, b] -= g * wj[f.j]


# ----------------------------------------------------------------------------
# noise estimates and thresholds  (Section "Thresholds")
# ----------------------------------------------------------------------------
def lower_median(x) -> float:
    """Element floor((N-1)/2) of the sorted values (the lower of the two middle ones)."""
    x = np.sort(np.asarray(x, dtype=np.float64).ravel())
    return float(x[(x.size - 1) // 2])


def sigma_mad(S, of_abs: int = 1) -> float:
    """1.4826 median(||S| - median|S||) as printed (of_abs=1), or the signed form
    1.4826 median|S - median S| (of_abs=0)."""
    x = np.asarray(S, dtype=np.float64).ravel()
    if of_abs:
        x = np.abs(x)
    med = lower_median(x)
    return 1.4826 * lower_median(np.abs(x - med))


def cap_K(params: Params) -> int:
    """K = max(64, 8 s)."""
    return max(64, 8 * params.s_budget)


def select_candidates(S, thr: float, K: int) -> np.ndarray:
    """Flat indices of the K largest |S_ab| among those with |S_ab| > thr, ordered by
    descending |S|, ties by ascending flat index (Algorithm 1, set Q)."""
    a = np.abs(np.asarray(S, dtype=np.float64)).ravel()
    with np.errstate(invalid="ignore"):
        idx = np.nonzero(a > thr)[0]
    order = np.lexsort((idx, -a[idx]))
    return idx[order][:K]


def decode_candidates(S, R, T, cand: np.ndarray, n1: int, n3: int):
    """U = candidates with S != 0 and S, R, T finite; their 0-based rounded
    coordinates from Eq. (recover).  Returns a list of (flat, i_hat, j_hat)."""
    p1 = (n1 - 1).bit_length() if n1 > 1 else 0
    p3 = (n3 - 1).bit_length() if n3 > 1 else 0
    Sf, Rf, Tf = (np.asarray(x, dtype=np.float64).ravel() for x in (S, R, T))
    out = []
    for f in cand:
        s, r_, t_ = Sf[f], Rf[f], Tf[f]
        if s == 0.0 or not (np.isfinite(s) and np.isfinite(r_) and np.isfinite(t_)):
            continue
        ih = np.rint((2.0 ** p1) * r_ / s) - 1.0
        jh = np.rint((2.0 ** p3) * t_ / s) - 1.0
        # keep the rounded index in integer range; far-off values can never reach C
        ih = int(max(min(ih, 2.0 ** 40), -(2.0 ** 40)))
        jh = int(max(min(jh, 2.0 ** 40), -(2.0 ** 40)))
        out.append((int(f), ih, jh))
    return out


def search_offsets(r: int):
    """Offsets (d_i, d_j), |d_i|,|d_j| <= r, by Chebyshev then Manhattan distance,
    ties by d_i then d_j."""
    offs = [(di, dj) for di in range(-r, r + 1) for dj in range(-r, r + 1)]
    offs.sort(key=lambda o: (max(abs(o[0]), abs(o[1])), abs(o[0]) + abs(o[1]), o[0], o[1]))
    return offs


def validate_entry(A, B, C, i: int, j: int, c_valid: float = 100.0):
    """gamma = A_i,* . B_*,j in FP64; accept iff |gamma - C_ij| > c eps sum_k|A_ik||B_kj|
    (Section "Validation").  Returns (accepted, gamma, tau_ij)."""
    a = np.asarray(A[i, :], dtype=np.float64)
    b = np.asarray(B[:, j], dtype=np.float64)
    gamma = float(np.dot(a, b))
    tau_ij = c_valid * EPS32 * float(np.dot(np.abs(a), np.abs(b)))
    cij = float(C[i, j])
    diff = abs(gamma - cij)
    return (diff > tau_ij), gamma, tau_ij


def localize_round(A, B, C, E, seed: int, rnd: int, m_b: int, r: int, F: List[Fault],
                   params: Params, tau: float, stats: Optional[dict] = None) -> List[Fault]:
    """One round of Algorithm 1.  E is the explicit error matrix (the sketch source);
    A, B, C feed the independent recomputation."""
    n1, n3 = E.shape
    h1, v1 = hash_round(seed, rnd, 0, n1, m_b)
    h2, v2 = hash_round(seed, rnd, 1, n3, m_b)
    S, R, T = moment_sketches(E, h1, v1, h2, v2, m_b)
    peel(S, R, T, F, h1, v1, h2, v2, n1, n3)
    sig = sigma_mad(S, params.mad_of_abs)
    tau_c = min(tau, 2.0 * sig)
    tau_d = max(n1, n3) * sig / max(float(r), 0.5)
    thr = max(tau_c, tau_d)
    K = cap_K(params)
    Q = select_candidates(S, thr, K)
    U = decode_candidates(S, R, T, Q, n1, n3)
    if stats is not None:
        stats.setdefault("rounds", []).append(
            dict(sigma_mad=sig, tau_c=tau_c, tau_d=tau_d, n_Q=len(Q), n_U=len(U),
                 S=S, R=R, T=T, h1=h1, h2=h2, candidates=list(U)))
    inF = {(f.i, f.j) for f in F}
    alive = list(U)
    for (di, dj) in search_offsets(r):
        if not alive:
            break
        still = []
        for (flat, ih, jh) in alive:
            i, j = ih + di, jh + dj
            if i < 0 or i >= n1 or j < 0 or j >= n3 or (i, j) in inF:
                still.append((flat, ih, jh))
                continue
            ok, gamma, _ = validate_entry(A, B, C, i, j, params.c_valid)
            if ok:
                cij = float(C[i, j])
                F.append(Fault(i, j, gamma - cij, gamma, cij, rnd, flat // m_b, flat % m_b))
                inF.add((i, j))
            else:
                still.append((flat, ih, jh))
        alive = still
    return F


def localize(A, B, C, seed: int, m_b: int, dtype: int, params: Params = None,
             E: Optional[np.ndarray] = None, stats: Optional[dict] = None) -> List[Fault]:
    """Localize part of Algorithm 2: k fresh rounds of Algorithm 1 at the caller's
    bucket count, carrying F.  Returns F sorted by (i, j)."""
    params = params or Params()
    A64, B64 = _f64(A), _f64(B)
    C = np.asarray(C)
    n1, n2 = A64.shape
    n3 = B64.shape[1]
    if E is None:
        E = A64 @ B64 - _f64(C)
    tau = analytic_tau(A64, B64, n2)
    r = params.radius
    if r < 0:
        # no calibration handed in: measure sigma_MAD on the first round's S
        # (Section "Calibration") and take the radius the budget asks for at m_b
        h1, v1 = hash_round(seed, 0, 0, n1, m_b)
        h2, v2 = hash_round(seed, 0, 1, n3, m_b)
        S0, _, _ = moment_sketches(E, h1, v1, h2, v2, m_b)
        sig0 = sigma_mad(S0, params.mad_of_abs)
        rms = rms_c_estimate(C)
        if not (np.isfinite(sig0) and sig0 > 0 and np.isfinite(rms) and rms > 0):
            sig0 = law_sigma(n1, n2, n3, dtype, 1.0, m_b)
            rms = 1.0
        r = min(params.r_max, radius_from_budget(index_budget(n1, n3, sig0, rms, params.rho_min)))
    if stats is not None:
        stats["radius"] = r
        stats["tau"] = tau
    F: List[Fault] = []
    for t in range(params.rounds):
        F = localize_round(A64, B64, C, E, seed, t, m_b, r, F, params, tau, stats)
    return sorted(F, key=lambda f: (f.i, f.j))


# ----------------------------------------------------------------------------
# sizing law and calibration plan  (Sections "Sketch Noise Sets the Bucket Count"
# and "Fault Magnitude, Calibration, and the Neighbourhood Search")
# ----------------------------------------------------------------------------
def c_f(dtype: int) -> float:
    """0.19 for BF16 operands, 1.76 x 0.19 for FP16 (the product, not its rounded print)."""
    return 0.19 if dtype == BF16 else 1.76 * 0.19


def law_sigma(n1, n2, n3, dtype, rms, m) -> float:
    """Eq. (sigma): c_f 2^-24 sqrt(n1 n3 n2) (n2/8192)^0.07 rms(C) / m."""
    return c_f(dtype) * 2.0 ** -24 * math.sqrt(float(n1) * n3 * n2) * (n2 / 8192.0) ** 0.07 * rms / m


def m_comb(params: Params) -> int:
    """ceil(max(3 c Delta, sqrt(3 c s))) with the collision constant c."""
    return int(math.ceil(max(3 * params.c_coll * params.delta_max,
                             math.sqrt(3 * params.c_coll * params.s_budget))))


def m_max(n1, n3) -> int:
    """max(16, floor(sqrt(n1 n3 / 16))): keeps 16 entries per bucket on average."""
    return max(16, math.isqrt((n1 * n3) // 16))


def m_mem(n2) -> int:
    """Largest m with 4 (3 m^2 + 6 m n2) bytes within 2 GiB."""
    lim = (1 << 31) // 4
    # 3 m^2 + 6 n2 m - lim <= 0
    m = int((-6 * n2 + math.sqrt(36.0 * n2 * n2 + 12.0 * lim)) / 6.0)
    while 3 * (m + 1) ** 2 + 6 * (m + 1) * n2 <= lim:
        m += 1
    while m > 0 and 3 * m * m + 6 * m * n2 > lim:
        m -= 1
    return m


def m_num(n1, n2, n3, dtype, params: Params, rho: float = 1.0) -> int:
    """Eq. (mnum) at delta = rho rms(C) and target budget B*."""
    x = max(n1, n3) / (params.b_star * rho) * law_sigma(n1, n2, n3, dtype, 1.0, 1.0)
    return int(math.ceil(x))


def m_start(n1, n2, n3, dtype, params: Params = None) -> int:
    """Eq. (mstart): min(max(m_comb, m_num, 16), max(m_comb, m_max))."""
    params = params or Params()
    mc = m_comb(params)
    return min(max(mc, m_num(n1, n2, n3, dtype, params), 16), max(mc, m_max(n1, n3)))


def rms_c_estimate(C) -> float:
    """rms of the finite entries of C taken at stride max(1, floor(n1 n3 / 65536)) from
    flat index 0, magnitudes clipped at 64 times their (lower) median."""
    flat = np.asarray(C).ravel()
    st = max(1, flat.size // 65536)
    x = np.abs(flat[::st].astype(np.float64))
    x = x[np.isfinite(x)]
    if x.size == 0:
        return float("nan")
    med = lower_median(x)
    x = np.minimum(x, 64.0 * med)
    return float(math.sqrt(np.mean(x * x)))


def index_budget(n1, n3, sigma, rms, rho_min) -> float:
    """B = max(n1,n3) sigma / (rho_min rms)."""
    return max(n1, n3) * sigma / (rho_min * rms)


def radius_from_budget(B: float) -> int:
    """r_B = 0 if B <= 0.05 else max(2, ceil(2.5 B))."""
    return 0 if B <= 0.05 else max(2, int(math.ceil(2.5 * B)))


def plan(n1, n2, n3, dtype, sigma_hat, rms_c, m_cur, params: Params = None):
    """Calibration plan: (m_loc, r, B) from the measured noise at bucket count m_cur."""
    params = params or Params()
    ok = all(np.isfinite(v) and v > 0 for v in (sigma_hat, rms_c))
    if not ok:
        sigma_hat = law_sigma(n1, n2, n3, dtype, 1.0, m_cur)
        rms_c = 1.0
    B = index_budget(n1, n3, sigma_hat, rms_c, params.rho_min)
    r_B = radius_from_budget(B)
    if r_B <= params.r_star:
        return m_cur, r_B, B
    grown = 16 * int(math.ceil(math.ceil(m_cur * r_B / params.r_star) / 16.0))
    m_loc = max(m_cur, min(grown, m_max(n1, n3), m_mem(n2)))
    Bp = B * m_cur / m_loc
    r = 0 if Bp <= 0.05 else min(params.r_max, max(2, int(math.ceil(2.5 * Bp))))
    return m_loc, r, B


def recalibrated_m(n1, n3, sigma_bar, rms_c, m_cur, params: Params = None) -> int:
    """m' = max(m_comb, 16, min(ceil(m B1 / B*), m_max)), B1 = max(n1,n3) sigma / rms."""
    params = params or Params()
    B1 = max(n1, n3) * sigma_bar / rms_c
    return max(m_comb(params), 16, min(int(math.ceil(m_cur * B1 / params.b_star)), m_max(n1, n3)))


# ----------------------------------------------------------------------------
# stateful probe  (Section "Calibration", paragraph "Recalibrating the probe";
# Section "Implementation": verdict accumulated into one flag per step)
# ----------------------------------------------------------------------------
@dataclass
class ProbeState:
    """What the probe keeps between calls: how many calls, how many it reported clean, the sum of
    sigma_hat over the clean ones, and the OR of the verdicts since the last reset."""
    calls: int = 0
    clean_calls: int = 0
    fired_any: int = 0
    first_fired_call: int = 0       # 1-based index of the first dirty call since the reset, 0 = none
    sigma_sum: float = 0.0

    def accumulate(self, r: ProbeResult) -> None:
        self.calls += 1
        if r.fired:
            if not self.fired_any:
                self.first_fired_call = self.calls
            self.fired_any = 1
        else:
            self.clean_calls += 1
            self.sigma_sum += float(np.float32(r.sigma_hat))

    def sigma_bar(self) -> float:
        return self.sigma_sum / self.clean_calls if self.clean_calls else float("nan")


def recalibration_due(calls: int) -> bool:
    """After 16 calls and then every 1024: taken as call counts 16, 1024, 2048, ..."""
    return calls == 16 or (calls > 16 and calls % 1024 == 0)


def recalibrate_probe(n1, n3, sigma_bar, rms_c, m_cur, params: Params = None):
    """(m', rebuild): m' from the averaged clean-call noise; the engine rebuilds at m' only when m'
    lies outside [m / 1.25, 1.25 m].  A noise or rms estimate that is not a positive finite number
    leaves m unchanged."""
    ok = all(math.isfinite(x) and x > 0 for x in (sigma_bar, rms_c))
    if not ok:
        return m_cur, False
    m_new = recalibrated_m(n1, n3, sigma_bar, rms_c, m_cur, params)
    return m_new, (m_new < m_cur / 1.25 or m_new > 1.25 * m_cur)


def measure_noise(A, B, C, seed: int, dtype: int, m0: int = 0, params: Params = None,
                  E: Optional[np.ndarray] = None) -> NoiseResult:
    """Run-time noise measurement: the hashed sum sketch S of round 0 at m0 (the law's
    starting bucket count when m0 = 0), both noise estimates, the strided rms of C,
    the normalized constant, and the plan that follows from them."""
    params = params or Params()
    A64, B64 = _f64(A), _f64(B)
    n1, n2 = A64.shape
    n3 = B64.shape[1]
    if m0 <= 0:
        m0 = m_start(n1, n2, n3, dtype, params)
    if E is None:
        E = A64 @ B64 - _f64(C)
    h1, v1 = hash_round(seed, 0, 0, n1, m0)
    h2, v2 = hash_round(seed, 0, 1, n3, m0)
    S, _, _ = moment_sketches(E, h1, v1, h2, v2, m0)
    s_clip = sigma_clip(S)
    s_mad = sigma_mad(S, params.mad_of_abs)
    rms = rms_c_estimate(C)
    if np.isfinite(rms) and rms > 0:
        c_hat = s_clip * m0 / (2.0 ** -24 * math.sqrt(float(n1) * n2 * n3) * rms)
    else:
        c_hat = float("nan")
    m_loc, r, Bv = plan(n1, n2, n3, dtype, s_clip, rms, m0, params)
    if np.isfinite(rms) and rms > 0 and np.isfinite(s_clip) and s_clip > 0:
        m_probe = recalibrated_m(n1, n3, s_clip, rms, m0, params)
    else:
        m_probe = m0
    return NoiseResult(s_clip, s_mad, rms, c_hat, Bv, m0, m_probe, m_loc, r)


# ----------------------------------------------------------------------------
# Algorithm 2 complete: exact scan, absolute repairs, apply, second probe
# (Section "Nonfinite and Out of Range Entries"; Algorithm 2)
# ----------------------------------------------------------------------------
FP32_MAX = float(np.finfo(np.float32).max)


def scan_out_of_range(C, K: int):
    """Coordinates of entries that are not finite or larger than fp32max/16 in magnitude, in
    row-major order, at most K of them."""
    C = np.asarray(C)
    with np.errstate(invalid="ignore"):
        bad = ~(np.abs(C.astype(np.float64)) <= FP32_MAX / 16.0)
    ii, jj = np.nonzero(bad)
    return [(int(i), int(j)) for i, j in zip(ii[:K], jj[:K])]


def apply_corrections(C, F: List[Fault]) -> np.ndarray:
    """C_ij <- delta for absolute entries (round < 0), C_ij <- C_ij + delta otherwise, in FP32."""
    out = np.array(C, dtype=np.float32, copy=True)
    for f in F:
        if f.round < 0:
            out[f.i, f.j] = np.float32(f.delta)
        else:
            out[f.i, f.j] = np.float32(np.float64(out[f.i, f.j]) + f.delta)
    return out


def verify_repair(A, B, C, seed: int, dtype: int, params: Params = None, m_b: int = 0):
    """Algorithm 2: probe; scan; absolute repairs held in C while the sketches are built; plan
    from sigma_MAD of a fresh S at the law's bucket count and the strided rms of C (unless m_b
    is given); k rounds of Algorithm 1; restore; apply; second probe.
    Returns (C_out, F sorted by (i, j), report dict)."""
    params = params or Params()
    A64, B64 = _f64(A), _f64(B)
    C = np.array(C, dtype=np.float32, copy=True)
    n1, n2 = A64.shape
    n3 = B64.shape[1]
    tau = analytic_tau(A64, B64, n2)
    AB = A64 @ B64
    first = probe_verdict(probe_sketch(AB - C.astype(np.float64)), tau, params, n_rows=n1)
    rep = dict(state=0, n_faults=0, n_absolute=0, m_loc=0, radius=0, first_probe=first, second_probe=None)
    if not first.fired:
        return C, [], rep
    K = cap_K(params)
    F: List[Fault] = []
    work = C.copy()
    for (i, j) in scan_out_of_range(C, K):
        gamma = float(np.dot(A64[i, :], B64[:, j]))
        F.append(Fault(i, j, gamma, gamma, float(C[i, j]), -1, -1, -1))
        work[i, j] = np.float32(gamma)
    rep["n_absolute"] = len(F)
    E = AB - work.astype(np.float64)
    r = params.radius
    if m_b <= 0:
        m0 = m_start(n1, n2, n3, dtype, params)
        h1, v1 = hash_round(seed, 0, 0, n1, m0)
        h2, v2 = hash_round(seed, 0, 1, n3, m0)
        S0, _, _ = moment_sketches(E, h1, v1, h2, v2, m0)
        m_b, r_plan, _ = plan(n1, n2, n3, dtype, sigma_mad(S0, params.mad_of_abs), rms_c_estimate(work), m0, params)
        if r < 0:
            r = r_plan
    if r < 0:
        h1, v1 = hash_round(seed, 0, 0, n1, m_b)
        h2, v2 = hash_round(seed, 0, 1, n3, m_b)
        S0, _, _ = moment_sketches(E, h1, v1, h2, v2, m_b)
        sig0, rms = sigma_mad(S0, params.mad_of_abs), rms_c_estimate(work)
        if not (np.isfinite(sig0) and sig0 > 0 and np.isfinite(rms) and rms > 0):
            sig0, rms = law_sigma(n1, n2, n3, dtype, 1.0, m_b), 1.0
        r = min(params.r_max, radius_from_budget(index_budget(n1, n3, sig0, rms, params.rho_min)))
    rep["m_loc"], rep["radius"] = m_b, r
    for t in range(params.rounds):
        # absolute entries are in F (never revisited) but are not peeled
        peeled = [f for f in F if f.round >= 0]
        known = [f for f in F if f.round < 0]
        Ft = list(peeled)
        Ft = _round_with_known(A64, B64, work, E, seed, t, m_b, r, Ft, known, params, tau)
        F = known + Ft
    F = sorted(F, key=lambda f: (f.i, f.j))
    C_out = apply_corrections(C, F)
    second = probe_verdict(probe_sketch(AB - C_out.astype(np.float64)), tau, params, n_rows=n1)
    rep["second_probe"] = second
    rep["n_faults"] = len(F)
    rep["state"] = 2 if second.fired else 1
    return C_out, F, rep


def _round_with_known(A64, B64, C, E, seed, rnd, m_b, r, F_finite, F_abs, params, tau):
    """One round of Algorithm 1 where F = F_finite + F_abs: only F_finite is peeled, both are
    skipped by the search."""
    n1, n3 = E.shape
    h1, v1 = hash_round(seed, rnd, 0, n1, m_b)
    h2, v2 = hash_round(seed, rnd, 1, n3, m_b)
    S, R, T = moment_sketches(E, h1, v1, h2, v2, m_b)
    peel(S, R, T, F_finite, h1, v1, h2, v2, n1, n3)
    sig = sigma_mad(S, params.mad_of_abs)
    thr = max(min(tau, 2.0 * sig), max(n1, n3) * sig / max(float(r), 0.5))
    U = decode_candidates(S, R, T, select_candidates(S, thr, cap_K(params)), n1, n3)
    inF = {(f.i, f.j) for f in F_finite} | {(f.i, f.j) for f in F_abs}
    alive = list(U)
    for (di, dj) in search_offsets(r):
        if not alive:
            break
        still = []
        for (flat, ih, jh) in alive:
            i, j = ih + di, jh + dj
            if i < 0 or i >= n1 or j < 0 or j >= n3 or (i, j) in inF:
                still.append((flat, ih, jh))
                continue
            ok, gamma, _ = validate_entry(A64, B64, C, i, j, params.c_valid)
            if ok:
                cij = float(C[i, j])
                F_finite.append(Fault(i, j, gamma - cij, gamma, cij, rnd, flat // m_b, flat % m_b))
                inF.add((i, j))
            else:
                still.append((flat, ih, jh))
        alive = still
    return F_finite
