"""Parity of the CUDA path (through the C ABI) with the CPU oracle, on the same seeded inputs.

Bar: bit-exact for integer work (hash tables, bucket assignment, planner integers, fired flag
and coordinate sets outside the detection margin); within 1e-5 of sum|A||B| for sketch values,
the probe residual and recovered magnitudes.
"""
import math

import numpy as np
import pytest
import torch

import oracle as O
from paper_2609_19758_b200 import build as B
from paper_2609_19758_b200 import fpsk, harness, workloads as W

pytestmark = pytest.mark.gpu
TOL = 1e-5


@pytest.fixture(scope="module", autouse=True)
def _lib():
    B.build()
    fpsk.lib()


def _to_dev(*ts):
    return [t.cuda() for t in ts]


def _case(kind, n1, n2, n3, dtype, seed, vendor=True):
    A, Bm = W.operands(kind, n1, n2, n3, dtype, seed)
    if vendor and n1 % 8 == 0 and n2 % 8 == 0 and n3 % 8 == 0:
        dA, dB = _to_dev(A, Bm)
        Cm = harness.vendor_gemm_fp32(dA, dB).cpu()
    else:
        Cm = W.cpu_fp32_product(A, Bm)
    return A, Bm, Cm


def _f64(t):
    return t.double().numpy()


def _run_probe(A, Bm, Cm, params=None, want_residual=True):
    dA, dB, dC = _to_dev(A, Bm, Cm)
    n1, n2 = A.shape
    n3 = Bm.shape[1]
    ws = fpsk.probe_workspace(n1, n2, n3)
    res = fpsk.new_probe_result()
    resid = torch.empty(n3, dtype=torch.float32, device="cuda") if want_residual else None
    fpsk.probe(dA, dB, dC, ws, res, resid, params)
    torch.cuda.synchronize()
    return fpsk.read_probe_result(res), (resid.cpu().numpy().astype(np.float64) if want_residual else None), ws


# ------------------------------------------------------------------ hash tables: bit exact
@pytest.mark.parametrize("seed,rnd,side,n,m_b", [(1, 0, 0, 1, 1), (7, 1, 1, 257, 17), (2 ** 40 + 3, 2, 0, 4096, 48),
                                                 (99, 0, 1, 16384, 4096), (12345678901234567, 5, 1, 11008, 1187)])
def test_hash_tables_bit_exact(seed, rnd, side, n, m_b):
    b, s = fpsk.hash_tables(seed, rnd, side, n, m_b)
    hb, hs = O.hash_round(seed, rnd, side, n, m_b)
    assert np.array_equal(b.cpu().numpy().astype(np.int64), hb)
    assert np.array_equal(s.cpu().numpy().astype(np.float64), hs)


# ------------------------------------------------------------------ probe
PROBE_SHAPES = [(1, 1, 1), (7, 5, 9), (33, 17, 40), (255, 256, 257), (256, 256, 256), (257, 255, 33),
                (1024, 512, 2048), (512, 4096, 1000), (2048, 1384, 4104)]


@pytest.mark.parametrize("shape", PROBE_SHAPES)
@pytest.mark.parametrize("dtype", [W.FP16, W.BF16])
def test_probe_residual_and_verdict(shape, dtype):
    n1, n2, n3 = shape
    A, Bm, Cm = _case("uniform" if dtype == W.FP16 else "gauss_scaled", n1, n2, n3, dtype, 5)
    A64, B64 = _f64(A), _f64(Bm)
    E = O.error_matrix(A64, B64, Cm.numpy())
    s_ref = O.probe_sketch(E)
    abs_j = O.abs_product(A64, B64).sum(axis=0)
    tau = O.analytic_tau(A64, B64, n2)
    got, resid, _ = _run_probe(A, Bm, Cm)
    assert got.status == 0
    assert np.all(np.abs(resid - s_ref) <= TOL * abs_j + 1e-30)
    assert got.tau == pytest.approx(tau, rel=1e-6)
    # the verdict formula applied to the GPU's own residual, in FP64
    v = O.probe_verdict(resid, tau, n_rows=n1)
    assert got.sigma_hat == pytest.approx(v.sigma_hat, rel=1e-4, abs=1e-30)
    assert got.thr == pytest.approx(v.thr, rel=1e-4, abs=1e-30)
    assert got.max_abs == pytest.approx(v.max_abs, rel=1e-6, abs=1e-30)
    assert got.nonfinite == 0
    if abs(v.max_abs - v.thr) > 1e-3 * v.thr:
        assert bool(got.fired) == v.fired
    if n3 >= 256:
        assert not got.fired and not O.probe_verdict(s_ref, tau, n_rows=n1).fired      # clean product


def test_probe_fires_on_faults_and_not_on_clean_with_the_oracle():
    n = 1024
    A, Bm, Cm = _case("gauss_scaled", n, n, n, W.BF16, 11)
    A64, B64 = _f64(A), _f64(Bm)
    tau = O.analytic_tau(A64, B64, n)
    rms = W.rms(Cm)
    AB = A64 @ B64
    for s in range(4):
        f = W.faults_additive(n, n, rms, s, 1, 0.02, 0.09, "small")
        Cf, ch = W.inject(Cm, f)
        got, resid, _ = _run_probe(A, Bm, Cf)
        ref = O.probe_verdict(O.probe_sketch(AB - Cf.double().numpy()), tau, n_rows=n)
        assert ref.fired and got.fired == 1
        assert got.argmax_col == ref.argmax_col == f[0].j
        assert got.max_abs == pytest.approx(abs(ch[0]), rel=0.05)


def test_probe_nonfinite_and_rejections():
    A, Bm, Cm = _case("uniform", 64, 64, 64, W.FP16, 3)
    Cn = Cm.clone()
    Cn[5, 7] = float("nan")
    got, _, _ = _run_probe(A, Bm, Cn)
    assert got.fired == 1 and got.nonfinite == 1
    Cn[5, 7] = float("inf")
    got, _, _ = _run_probe(A, Bm, Cn)
    assert got.fired == 1 and got.nonfinite == 1
    dA, dB, dC = _to_dev(A, Bm, Cm)
    ws = fpsk.probe_workspace(64, 64, 64)
    res = fpsk.new_probe_result()
    with pytest.raises(fpsk.FpskError) as e:
        fpsk.probe(dA, dB, dC, ws, res, c_is_fp32=False)        # a narrowed C is rejected
    assert e.value.status == fpsk.ERR_DTYPE
    with pytest.raises(fpsk.FpskError) as e:
        fpsk.probe(dA, dB, dC, ws[:512], res)
    assert e.value.status == fpsk.ERR_WORKSPACE


def test_probe_strided_views_and_determinism():
    A, Bm, Cm = _case("uniform", 96, 80, 72, W.FP16, 8, vendor=False)
    dA, dB, dC = _to_dev(A, Bm, Cm)
    # embed in wider buffers: leading dimensions larger than the column counts, odd offsets
    bigA = torch.zeros(96, 91, dtype=dA.dtype, device="cuda"); bigA[:, 3:83] = dA
    bigB = torch.zeros(80, 104, dtype=dB.dtype, device="cuda"); bigB[:, 8:80] = dB
    bigC = torch.full((96, 77), 9.0, device="cuda"); bigC[:, 1:73] = dC
    ws = fpsk.probe_workspace(96, 80, 72)
    res = fpsk.new_probe_result()
    r1 = torch.empty(72, device="cuda"); r2 = torch.empty(72, device="cuda"); r3 = torch.empty(72, device="cuda")
    fpsk.probe(dA, dB, dC, ws, res, r1)
    fpsk.probe(bigA[:, 3:83], bigB[:, 8:80], bigC[:, 1:73], ws, res, r2)
    fpsk.probe(dA, dB, dC, ws, res, r3)
    torch.cuda.synchronize()
    assert torch.equal(r1, r3)                          # bit-identical rerun
    s_ref = O.probe_sketch(O.error_matrix(_f64(A), _f64(Bm), Cm.numpy()))
    abs_j = O.abs_product(_f64(A), _f64(Bm)).sum(axis=0)
    assert np.all(np.abs(r2.cpu().numpy() - s_ref) <= TOL * abs_j)


def test_probe_host_entry_point():
    A, Bm, Cm = _case("uniform", 256, 256, 256, W.FP16, 2)
    rms = W.rms(Cm)
    f = W.faults_additive(256, 256, rms, 1, 1, 0.5, 0.5, "typical")
    Cf, _ = W.inject(Cm, f)
    ws = fpsk.probe_host_workspace(256, 256, 256)
    clean = fpsk.probe_host(A.pin_memory(), Bm.pin_memory(), Cm.pin_memory(), ws)
    dirty = fpsk.probe_host(A.pin_memory(), Bm.pin_memory(), Cf.pin_memory(), ws)
    assert clean.fired == 0 and dirty.fired == 1 and dirty.argmax_col == f[0].j


# ------------------------------------------------------------------ sketches
def _sketch_parity(A, Bm, Cm, seed, rnd, m_b, exact=False):
    dA, dB, dC = _to_dev(A, Bm, Cm)
    n1, n2 = A.shape
    n3 = Bm.shape[1]
    ws = fpsk.workspace(n1, n2, n3, m_b)
    S, R, T = fpsk.sketches(dA, dB, dC, seed, rnd, m_b, ws)
    S2, _, _ = fpsk.sketches(dA, dB, dC, seed, rnd, m_b, ws, moments=False)
    torch.cuda.synchronize()
    A64, B64 = _f64(A), _f64(Bm)
    E = O.error_matrix(A64, B64, Cm.numpy())
    h1, v1 = O.hash_round(seed, rnd, 0, n1, m_b)
    h2, v2 = O.hash_round(seed, rnd, 1, n3, m_b)
    So, Ro, To = O.moment_sketches(E, h1, v1, h2, v2, m_b)
    ABS = O.abs_sketch(O.abs_product(A64, B64), h1, h2, m_b)
    for g, o in ((S, So), (R, Ro), (T, To), (S2, So)):
        g = g.cpu().numpy().astype(np.float64)
        if exact:
            assert np.array_equal(g, o)
        else:
            assert np.all(np.abs(g - o) <= TOL * ABS + 1e-30)
    return S, So


@pytest.mark.parametrize("shape,m_b", [((16, 12, 16), 4), ((7, 5, 9), 3), ((13, 16, 6), 1), ((33, 40, 65), 17)])
def test_sketches_exact_on_integer_inputs(shape, m_b):
    """Small integers and dyadic weights: every FP32 sum is exact, so the compressed-operand
    sketch on the GPU equals the explicit-E sketch of the oracle bit for bit."""
    n1, n2, n3 = shape
    A, Bm = W.operands("integer", n1, n2, n3, W.FP16, 4, lim=8)
    Cm = W.cpu_fp32_product(A, Bm)
    Cm[n1 // 2, n3 // 3] += 5.0
    Cm[0, n3 - 1] -= 3.0
    for rnd in range(2):
        _sketch_parity(A, Bm, Cm, 77, rnd, m_b, exact=True)


@pytest.mark.parametrize("shape,m_b,dtype", [((255, 256, 257), 16, W.FP16), ((256, 256, 256), 48, W.BF16),
                                             ((1024, 520, 768), 17, W.BF16), ((512, 1024, 2048), 200, W.FP16),
                                             ((2048, 1024, 1024), 256, W.BF16), ((64, 64, 64), 64, W.FP16)])
def test_sketches_within_tolerance(shape, m_b, dtype):
    n1, n2, n3 = shape
    A, Bm, Cm = _case("uniform" if dtype == W.FP16 else "gauss_scaled", n1, n2, n3, dtype, 9)
    rms = W.rms(Cm)
    Cf, _ = W.inject(Cm, W.faults_additive(n1, n3, rms, 3, 4, 0.02, 1.0, "small"))
    _sketch_parity(A, Bm, Cf, 2024, 1, m_b)


# ------------------------------------------------------------------ noise measurement
@pytest.mark.parametrize("n,dtype,kind", [(256, W.FP16, "uniform"), (1024, W.BF16, "gauss_scaled"), (1024, W.FP16, "gauss")])
def test_measure_noise_matches_oracle(n, dtype, kind):
    A, Bm, Cm = _case(kind, n, n, n, dtype, 13)
    dA, dB, dC = _to_dev(A, Bm, Cm)
    p = fpsk.default_params()
    po = O.Params()
    ws = fpsk.workspace(n, n, n, 0, p)
    got = fpsk.measure_noise(dA, dB, dC, 5, ws, 0, p)
    ref = O.measure_noise(_f64(A), _f64(Bm), Cm.numpy(), 5, dtype, 0, po)
    assert got.m0 == ref.m0
    assert got.rms_c == pytest.approx(ref.rms_c, rel=1e-5)
    # the GPU estimate contains the verifier's own FP32 rounding on top of the GEMM's.  Observed ratios on
    # these shapes: sigma_clip 1.19 / 1.03 / 1.02, sigma_MAD 1.05 / 1.02 / 1.04 (largest at n = 256, where
    # the GEMM's own noise is smallest)
    print("sigma_clip gpu/oracle", got.sigma_clip / ref.sigma_clip, "sigma_mad gpu/oracle", got.sigma_mad / ref.sigma_mad)
    assert 0.97 * ref.sigma_clip <= got.sigma_clip <= 1.3 * ref.sigma_clip
    assert 0.97 * ref.sigma_mad <= got.sigma_mad <= 1.3 * ref.sigma_mad
    # and so the plan drawn from it is the oracle's
    assert (got.m_loc, got.radius) == (ref.m_loc, ref.radius)
    # the plan is the oracle's plan for the GPU's own measurements (same scalar rule)
    ml, r, Bv = O.plan(n, n, n, dtype, got.sigma_clip, got.rms_c, got.m0, po)
    assert (got.m_loc, got.radius) == (ml, r)
    assert got.m_probe == O.recalibrated_m(n, n, got.sigma_clip, got.rms_c, got.m0, po)
    assert got.c_hat == pytest.approx(got.sigma_clip * got.m0 / (2.0 ** -24 * n ** 1.5 * got.rms_c), rel=1e-9)


def test_estimators_on_a_known_sketch():
    """sigma_clip / sigma_MAD kernels against the oracle's estimators on the same S."""
    n = 512
    A, Bm, Cm = _case("gauss", n, n, n, W.BF16, 21)
    dA, dB, dC = _to_dev(A, Bm, Cm)
    for m0, mad_of_abs in ((48, 1), (37, 0), (128, 1)):
        p = fpsk.default_params(mad_of_abs=mad_of_abs)
        ws = fpsk.workspace(n, n, n, m0, p)
        got = fpsk.measure_noise(dA, dB, dC, 3, ws, m0, p)
        S, _, _ = fpsk.sketches(dA, dB, dC, 3, 0, m0, ws, moments=False)
        Sn = S.cpu().numpy().astype(np.float64)
        assert got.sigma_clip == pytest.approx(O.sigma_clip(Sn), rel=1e-5)
        assert got.sigma_mad == pytest.approx(O.sigma_mad(Sn.astype(np.float32).astype(np.float64), mad_of_abs), rel=1e-5)


# ------------------------------------------------------------------ localization
def _check_localize(A, Bm, Cm, faults, changes, seed, m_b, params, oparams, dtype, expect_all=True):
    dA, dB, dC = _to_dev(A, Bm, Cm)
    n1, n2 = A.shape
    n3 = Bm.shape[1]
    ws = fpsk.workspace(n1, n2, n3, m_b, params)
    got = fpsk.localize(dA, dB, dC, seed, m_b, ws, params)
    A64, B64 = _f64(A), _f64(Bm)
    ref = O.localize(A64, B64, Cm.numpy(), seed, m_b, dtype, oparams)
    gset = {(f.i, f.j) for f in got}
    rset = {(f.i, f.j) for f in ref}
    injected = {(f.i, f.j) for f in faults}
    assert gset <= injected and rset <= injected            # zero false positives on both sides
    assert gset == rset
    if expect_all:
        assert gset == injected
    rmap = {(f.i, f.j): f for f in ref}
    for f in got:
        a = np.abs(A64[f.i, :]) @ np.abs(B64[:, f.j])
        o = rmap[(f.i, f.j)]
        assert abs(f.delta - o.delta) <= TOL * a
        assert abs(f.recompute - o.recompute) <= TOL * a
        assert f.c_value == o.c_value
        h1, _ = O.hash_round(seed, f.round, 0, n1, m_b)
        h2, _ = O.hash_round(seed, f.round, 1, n3, m_b)
        assert (f.bucket_a, f.bucket_b) == (h1[f.i], h2[f.j])          # bucket assignment
    want = {(x.i, x.j): -c for x, c in zip(faults, changes)}
    for f in got:
        assert f.delta == pytest.approx(want[(f.i, f.j)], abs=1e-4 * max(1.0, abs(want[(f.i, f.j)])))
    return got


def test_localize_small_square_fp16_config():
    """256^3 FP16, U(-1,1): one clean product and three products with one fault of 0.5 rms."""
    n = 256
    A, Bm, Cm = _case("uniform", n, n, n, W.FP16, 1)
    p = fpsk.default_params(s_budget=1, delta_max=1)
    po = O.Params(s_budget=1, delta_max=1)
    dA, dB, dC = _to_dev(A, Bm, Cm)
    ws = fpsk.workspace(n, n, n, 0, p)
    nz = fpsk.measure_noise(dA, dB, dC, 7, ws, 0, p)
    assert nz.m0 == 16
    p.radius = nz.radius
    po.radius = nz.radius
    _check_localize(A, Bm, Cm, [], [], 7, nz.m_loc, p, po, W.FP16)          # clean: nothing reported
    rms = W.rms(Cm)
    for s in (1, 2, 3):
        f = W.faults_additive(n, n, rms, s, 1, 0.5, 0.5, "typical")
        Cf, ch = W.inject(Cm, f)
        got = _check_localize(A, Bm, Cf, f, ch, 7, nz.m_loc, p, po, W.FP16)
        assert len(got) == 1


def test_localize_exact_integer_multi_fault_peeling():
    n1, n2, n3, m_b = 64, 16, 48, 6
    A, Bm = W.operands("integer", n1, n2, n3, W.FP16, 31, lim=8)
    Cm = W.cpu_fp32_product(A, Bm)
    coords = [(5, 1), (5, 9), (5, 30), (17, 9), (28, 3), (2, 22), (63, 47), (0, 0)]
    faults = [W.InjectedFault(i, j, "add", 3.0 + t, "typical") for t, (i, j) in enumerate(coords)]
    Cf, ch = W.inject(Cm, faults)
    p = fpsk.default_params(radius=1, rounds=6)
    po = O.Params(radius=1, rounds=6)
    got = _check_localize(A, Bm, Cf, faults, ch, 2024, m_b, p, po, W.FP16, expect_all=False)
    for f in got:
        assert f.delta == -(3.0 + coords.index((f.i, f.j)))             # exact magnitudes


def test_localize_radius_from_first_round_when_not_given():
    n = 512
    A, Bm, Cm = _case("gauss_scaled", n, n, n, W.BF16, 17)
    rms = W.rms(Cm)
    f = W.faults_additive(n, n, rms, 2, 4, 0.05, 0.09, "small")
    Cf, ch = W.inject(Cm, f)
    p = fpsk.default_params(s_budget=4)
    po = O.Params(s_budget=4)
    _check_localize(A, Bm, Cf, f, ch, 3, 128, p, po, W.BF16)


def test_localize_capacity_and_bucket_errors():
    n = 128
    A, Bm, Cm = _case("uniform", n, n, n, W.FP16, 6)
    rms = W.rms(Cm)
    f = W.faults_additive(n, n, rms, 1, 3, 1.0, 1.0, "typical")
    Cf, _ = W.inject(Cm, f)
    dA, dB, dC = _to_dev(A, Bm, Cf)
    p = fpsk.default_params(radius=1)
    ws = fpsk.workspace(n, n, n, 32, p)
    with pytest.raises(fpsk.FpskError) as e:
        fpsk.localize(dA, dB, dC, 1, 32, ws, p, capacity=1)
    assert e.value.status == fpsk.ERR_CAPACITY
    with pytest.raises(fpsk.FpskError) as e:
        fpsk.localize(dA, dB, dC, 1, 64, ws, p)                         # workspace sized for 32
    assert e.value.status == fpsk.ERR_WORKSPACE


def test_a_device_wait_that_runs_out_reports_timeout_and_leaves_the_context_usable():
    """Every device-side wait of the library is bounded; this drives the give-up path with a short limit
    (a flag that nothing sets), then checks that the same stream still runs a probe."""
    flag = torch.zeros(1, dtype=torch.int32, device="cuda")
    res = fpsk.new_probe_result()
    fpsk.selftest_bounded_wait(flag, res)
    torch.cuda.synchronize()
    assert fpsk.read_probe_result(res).status == fpsk.ERR_TIMEOUT
    flag.fill_(1)
    fpsk.selftest_bounded_wait(flag, res)
    torch.cuda.synchronize()
    assert fpsk.read_probe_result(res).status == 0
    A, Bm, Cm = _case("uniform", 64, 64, 64, W.FP16, 3)
    got, _, _ = _run_probe(A, Bm, Cm)
    assert got.status == 0 and got.fired == 0


# ------------------------------------------------------------------ the ordered search over the hits (device walk)
@pytest.mark.parametrize("m_b,radius,tc", [(12, 3, 0), (24, 2, 0), (384, 4, 1)])
def test_localize_clustered_faults_equal_the_oracle_round_by_round(m_b, radius, tc):
    """Many faults, several of them neighbours (one bucket's window then holds several true entries, and the same
    entry lies in the windows of several buckets), few buckets (collisions, so later rounds and the peeling matter):
    the fault list must be the oracle's entry by entry - coordinates, the round and bucket of discovery, magnitudes -
    which pins the order of the walk over the hits, the one-accept-per-bucket rule and the membership test in F."""
    n1, n2, n3 = (96, 24, 80) if not tc else (768, 64, 640)
    A, Bm = W.operands("integer", n1, n2, n3, W.FP16, 77, lim=6)
    Cm = W.cpu_fp32_product(A, Bm)
    g = np.random.default_rng(m_b * 31 + radius)
    coords = set()
    for _ in range(9):                                   # nine clusters of up to four adjacent entries
        i, j = int(g.integers(1, n1 - 2)), int(g.integers(1, n3 - 2))
        for (di, dj) in [(0, 0), (0, 1), (1, 0), (1, 1)][: int(g.integers(1, 5))]:
            coords.add((i + di, j + dj))
    coords = sorted(coords)
    faults = [W.InjectedFault(i, j, "add", float(2 + (t % 7)) * (1 if t % 2 else -1), "typical") for t, (i, j) in enumerate(coords)]
    Cf, _ = W.inject(Cm, faults)
    p = fpsk.default_params(radius=radius, rounds=5, s_budget=len(coords), tensor_cores=tc)
    po = O.Params(radius=radius, rounds=5, s_budget=len(coords))
    ws = fpsk.workspace(n1, n2, n3, m_b, p)
    got = fpsk.localize(A.cuda(), Bm.cuda(), Cf.cuda(), 99, m_b, ws, p)
    ref = O.localize(_f64(A), _f64(Bm), Cf.numpy(), 99, m_b, W.FP16, po)
    key = lambda f: (f.i, f.j, f.round, f.bucket_a, f.bucket_b, f.delta, f.c_value)
    assert [key(f) for f in got] == [key(f) for f in ref]
    assert {(f.i, f.j) for f in got} <= set(coords) and len(got) >= len(coords) // 2
    # and again on the same workspace: nothing of the first call's device lists survives into the second
    again = fpsk.localize(A.cuda(), Bm.cuda(), Cf.cuda(), 99, m_b, ws, p)
    assert [key(f) for f in again] == [key(f) for f in got]


def test_localize_reports_overflow_of_the_hit_list():
    """A corrupted block larger than the hit list of a round (2048 entries): the call says so (FPSK_ERR_CAPACITY)
    instead of returning a silently shortened list, and what it does return are true entries."""
    n1, n2, n3, m_b = 256, 32, 256, 16
    A, Bm = W.operands("integer", n1, n2, n3, W.FP16, 5, lim=6)
    Cm = W.cpu_fp32_product(A, Bm)
    Cf = Cm.clone()
    Cf[100:160, 100:160] += 5.0                          # 3600 faulty entries in one 60 x 60 block
    p = fpsk.default_params(radius=16, rounds=1, s_budget=128)
    ws = fpsk.workspace(n1, n2, n3, m_b, p)
    with pytest.raises(fpsk.FpskError) as e:
        fpsk.localize(A.cuda(), Bm.cuda(), Cf.cuda(), 3, m_b, ws, p)
    assert e.value.status == fpsk.ERR_CAPACITY
