"""Parity of the S only probe with a cached B side (Section "The Cheap S Only Probe") with the oracle.

S within 1e-5 of the bucket's sum of sum_k |A_ik||B_kj|; the verdict through the oracle's rule applied
to the GPU's own S; bit-exact on integer products; the cache key logic on the device path.
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


def _f64(t):
    return t.double().numpy()


def _case(kind, n1, n2, n3, dtype, seed):
    A, Bm = W.operands(kind, n1, n2, n3, dtype, seed)
    if n1 % 8 == 0 and n2 % 8 == 0 and n3 % 8 == 0:
        Cm = harness.vendor_gemm_fp32(A.cuda(), Bm.cuda()).cpu()
    else:
        Cm = W.cpu_fp32_product(A, Bm)
    return A, Bm, Cm


def _run(hp, A, Bm, Cm, version=0, params=None):
    m = hp.n_buckets
    res = fpsk.new_probe_result()
    S = torch.full((m, m), float("nan"), dtype=torch.float32, device="cuda")
    hp(A, Bm, Cm, res, b_version=version, S=S, params=params)
    torch.cuda.synchronize()
    return fpsk.read_probe_result(res), S.cpu().numpy().astype(np.float64)


SHAPES = [
    # (n1, n2, n3, m)   bulk-copy path: n2 % 8 == 0, n3 % 4 == 0
    (64, 64, 64, 4), (256, 256, 256, 16), (512, 2056, 1028, 48), (1024, 512, 2048, 64), (1000, 4104, 1500, 100),
    (2048, 1384, 4104, 256), (300, 8, 4, 7), (96, 4096, 96, 1),
    # plain path: odd sizes
    (7, 5, 9, 3), (33, 17, 40, 5), (255, 256, 257, 16), (257, 255, 33, 48),
]


@pytest.mark.parametrize("shape", SHAPES)
@pytest.mark.parametrize("dtype", [W.FP16, W.BF16])
@pytest.mark.parametrize("tensor_cores,scale_cap", [(0, 0), (1, 0), (0, 1)])
def test_sketch_and_verdict(shape, dtype, tensor_cores, scale_cap):
    n1, n2, n3, m = shape
    A, Bm, Cm = _case("uniform" if dtype == W.FP16 else "gauss_scaled", n1, n2, n3, dtype, 5)
    A64, B64 = _f64(A), _f64(Bm)
    ref, S_ref = O.probe_hashed(A64, B64, Cm.numpy(), 21, 4, m, O.Params(scale_cap=scale_cap))
    h1, _ = O.hash_round(21, 4, 0, n1, m)
    h2, _ = O.hash_round(21, 4, 1, n3, m)
    denom = O.abs_sketch(O.abs_product(A64, B64), h1, h2, m)
    hp = fpsk.HashedProbe(n1, n2, n3, m, seed=21, rnd=4)
    got, S = _run(hp, A.cuda(), Bm.cuda(), Cm.cuda(), params=fpsk.default_params(tensor_cores=tensor_cores, scale_cap=scale_cap))
    assert got.status == 0
    assert np.all(np.abs(S - S_ref) <= TOL * denom + 1e-30)
    assert got.tau == pytest.approx(ref.tau, rel=1e-6)
    # the rule on the GPU's own S: the printed one, or with the cap widened by the root of the bucket population
    v = O.probe_verdict(S.ravel(), ref.tau, n_rows=n1 * n3 / float(m * m) if scale_cap else 1)
    assert got.sigma_hat == pytest.approx(v.sigma_hat, rel=1e-4, abs=1e-30)
    assert got.thr == pytest.approx(v.thr, rel=1e-4, abs=1e-30)
    assert got.max_abs == pytest.approx(v.max_abs, rel=1e-6, abs=1e-30)
    assert got.argmax_col == v.argmax_col
    assert got.nonfinite == 0
    if abs(v.max_abs - v.thr) > 1e-3 * v.thr:
        assert bool(got.fired) == v.fired


@pytest.mark.parametrize("shape", [(96, 64, 80, 8), (512, 2048, 1024, 32), (130, 72, 100, 5), (31, 9, 27, 4),
                                   (640, 1000, 768, 200)])
@pytest.mark.parametrize("tensor_cores", [0, 1])
def test_integer_products_are_bit_exact(shape, tensor_cores):
    n1, n2, n3, m = shape
    A, Bm = W.operands("integer", n1, n2, n3, W.FP16, 5)
    Cm = W.cpu_fp32_product(A, Bm)
    Cm[n1 // 3, n3 // 2] += 3.0
    Cm[n1 - 1, 0] -= 5.0
    ref, S_ref = O.probe_hashed(_f64(A), _f64(Bm), Cm.numpy(), 11, 7, m)
    hp = fpsk.HashedProbe(n1, n2, n3, m, seed=11, rnd=7)
    got, S = _run(hp, A.cuda(), Bm.cuda(), Cm.cuda(), params=fpsk.default_params(tensor_cores=tensor_cores))
    assert np.array_equal(S, S_ref)
    assert got.fired == 1 and ref.fired and got.argmax_col == ref.argmax_col and got.max_abs == ref.max_abs


def test_detection_agrees_with_the_oracle_on_small_faults():
    n, m = 1024, 64
    A, Bm, Cm = _case("gauss_scaled", n, n, n, W.BF16, 11)
    A64, B64 = _f64(A), _f64(Bm)
    rms = W.rms(Cm)
    hp = fpsk.HashedProbe(n, n, n, m, seed=3, rnd=0)
    dA, dB = A.cuda(), Bm.cuda()
    got, _ = _run(hp, dA, dB, Cm.cuda())
    ref, _ = O.probe_hashed(A64, B64, Cm.numpy(), 3, 0, m)
    assert not ref.fired and got.fired == 0
    h1, _ = O.hash_round(3, 0, 0, n, m)
    h2, _ = O.hash_round(3, 0, 1, n, m)
    for s in range(4):
        f = W.faults_additive(n, n, rms, s, 1, 0.02, 0.09, "small")
        Cf, ch = W.inject(Cm, f)
        got, _ = _run(hp, dA, dB, Cf.cuda())
        ref, _ = O.probe_hashed(A64, B64, Cf.numpy(), 3, 0, m)
        assert ref.fired and got.fired == 1
        assert got.argmax_col == ref.argmax_col == int(h1[f[0].i]) * m + int(h2[f[0].j])
    assert hp.side.rebuilds == 1                      # one B side served every call


def test_nonfinite_entries_fire():
    A, Bm, Cm = _case("uniform", 128, 64, 128, W.FP16, 3)
    hp = fpsk.HashedProbe(128, 64, 128, 8, seed=1)
    for bad in (float("nan"), float("inf"), float("-inf")):
        Cn = Cm.clone()
        Cn[5, 7] = bad
        got, S = _run(hp, A.cuda(), Bm.cuda(), Cn.cuda())
        assert got.fired == 1 and got.nonfinite == 1 and got.status == 0
        assert np.count_nonzero(~np.isfinite(S)) == 1


def test_cache_is_keyed_on_identity_and_version():
    n1, n2, n3, m = 256, 128, 192, 16
    A, Bm, Cm = _case("gauss_scaled", n1, n2, n3, W.BF16, 9)
    dA, dB, dC = A.cuda(), Bm.cuda(), Cm.cuda()
    hp = fpsk.HashedProbe(n1, n2, n3, m, seed=5)
    assert not hp.matches(dB, 0)
    r0, S0 = _run(hp, dA, dB, dC, version=0)
    assert hp.matches(dB, 0) and hp.side.rebuilds == 1
    before = fpsk.launch_count()
    r1, S1 = _run(hp, dA, dB, dC, version=0)
    per_call = fpsk.launch_count() - before
    assert hp.side.rebuilds == 1 and np.array_equal(S0, S1)         # cached: same result, nothing rebuilt
    assert per_call == 3                                             # row-bucket sums + fold, contraction, combine + verdict
    # an in-place update of B with a new version rebuilds; the product no longer matches C
    dB.mul_(2.0)
    r2, S2 = _run(hp, dA, dB, dC, version=1)
    assert hp.side.rebuilds == 2 and r2.fired == 1
    ref, S_ref = O.probe_hashed(_f64(A), 2.0 * _f64(Bm), Cm.numpy(), 5, 0, m)
    h1, _ = O.hash_round(5, 0, 0, n1, m)
    h2, _ = O.hash_round(5, 0, 1, n3, m)
    denom = O.abs_sketch(O.abs_product(_f64(A), 2.0 * _f64(Bm)), h1, h2, m)
    assert np.all(np.abs(S2 - S_ref) <= TOL * denom)
    # another tensor with the same contents is another identity
    dB2 = dB.clone()
    _run(hp, dA, dB2, dC, version=1)
    assert hp.side.rebuilds == 3


def test_rejections():
    A, Bm, Cm = _case("uniform", 64, 64, 64, W.FP16, 3)
    hp = fpsk.HashedProbe(64, 64, 64, 8, seed=1)
    res = fpsk.new_probe_result()
    with pytest.raises(fpsk.FpskError) as e:
        hp(A.cuda(), Bm.cuda(), Cm.cuda(), res, c_is_fp32=False)
    assert e.value.status == fpsk.ERR_DTYPE
    assert hp.side.rebuilds == 0


def test_reruns_are_bit_identical_and_paths_agree():
    n1, n2, n3, m = 1536, 1024, 2048, 96
    A, Bm, Cm = _case("gauss_scaled", n1, n2, n3, W.FP16, 4)
    dA, dB, dC = A.cuda(), Bm.cuda(), Cm.cuda()
    hp = fpsk.HashedProbe(n1, n2, n3, m, seed=8, rnd=2)
    r0, S0 = _run(hp, dA, dB, dC)
    for _ in range(3):
        r, S = _run(hp, dA, dB, dC)
        assert np.array_equal(S, S0) and r.sigma_hat == r0.sigma_hat and r.thr == r0.thr
    # a view with an odd column offset takes the plain-load path: same sketch within rounding
    big = torch.zeros(n1, n2 + 8, dtype=dA.dtype, device="cuda")
    big[:, 1:n2 + 1] = dA
    hp2 = fpsk.HashedProbe(n1, n2, n3, m, seed=8, rnd=2)
    r2, S2 = _run(hp2, big[:, 1:n2 + 1], dB, dC)
    h1, _ = O.hash_round(8, 2, 0, n1, m)
    h2, _ = O.hash_round(8, 2, 1, n3, m)
    denom = O.abs_sketch(O.abs_product(_f64(A), _f64(Bm)), h1, h2, m)
    assert np.all(np.abs(S2 - S0) <= 2 * TOL * denom)
    assert r2.tau == r0.tau


# ---------------------------------------------------------------- state across calls, graph replay
def test_state_accumulates_like_the_oracle():
    n1, n2, n3, m = 512, 256, 512, 32
    A, Bm, Cm = _case("gauss_scaled", n1, n2, n3, W.BF16, 13)
    Cf = Cm.clone()
    Cf[17, 300] += 1.0
    dA, dB, dC, dF = A.cuda(), Bm.cuda(), Cm.cuda(), Cf.cuda()
    hp = fpsk.HashedProbe(n1, n2, n3, m, seed=9)
    res = fpsk.new_probe_result()
    state = fpsk.new_probe_state()
    ref = O.ProbeState()
    for which in (0, 0, 1, 0, 1, 0, 0):
        hp(dA, dB, dF if which else dC, res, state=state)
        torch.cuda.synchronize()
        r = fpsk.read_probe_result(res)
        assert r.fired == which
        ref.accumulate(O.ProbeResult(bool(r.fired), bool(r.nonfinite), r.argmax_col, r.max_abs, r.sigma_hat, r.thr, r.tau))
    got = fpsk.read_probe_state(state)
    assert (got.calls, got.clean_calls, got.fired_any, got.first_fired_call) == (7, 5, 1, 3)
    assert (got.calls, got.clean_calls, got.fired_any, got.first_fired_call) == \
           (ref.calls, ref.clean_calls, ref.fired_any, ref.first_fired_call)
    assert got.sigma_sum == ref.sigma_sum                       # same values added in the same order, in FP64
    # the same bookkeeping for the column-sum probe, through the stand-alone kernel
    fpsk.reset_probe_state(state)
    pws = fpsk.probe_workspace(n1, n2, n3)
    ref = O.ProbeState()
    for which in (1, 0, 0):
        fpsk.probe(dA, dB, dF if which else dC, pws, res)
        fpsk.probe_accumulate(res, state)
        torch.cuda.synchronize()
        r = fpsk.read_probe_result(res)
        ref.accumulate(O.ProbeResult(bool(r.fired), bool(r.nonfinite), r.argmax_col, r.max_abs, r.sigma_hat, r.thr, r.tau))
    got = fpsk.read_probe_state(state)
    assert (got.calls, got.clean_calls, got.fired_any, got.first_fired_call, got.sigma_sum) == \
           (ref.calls, ref.clean_calls, ref.fired_any, ref.first_fired_call, ref.sigma_sum)
    assert (got.calls, got.fired_any, got.first_fired_call) == (3, 1, 1)


def test_probe_replays_from_a_cuda_graph():
    """One host read per step: the captured probe accumulates its verdicts and its noise on the device."""
    n1, n2, n3, m = 1024, 512, 1024, 64
    A, Bm, Cm = _case("gauss_scaled", n1, n2, n3, W.FP16, 21)
    dA, dB, dC = A.cuda(), Bm.cuda(), Cm.cuda().clone()
    hp = fpsk.HashedProbe(n1, n2, n3, m, seed=4)
    res = fpsk.new_probe_result()
    S = torch.zeros(m, m, dtype=torch.float32, device="cuda")
    state = fpsk.new_probe_state()
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        hp(dA, dB, dC, res, S=S)                     # builds the B side and sets kernel attributes outside the capture
    side.synchronize()
    r0 = fpsk.read_probe_result(res)
    S0 = S.cpu().numpy().copy()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        hp(dA, dB, dC, res, S=S, state=state)
    rebuilds = hp.side.rebuilds
    for _ in range(5):
        g.replay()
    torch.cuda.synchronize()
    st = fpsk.read_probe_state(state)
    assert (st.calls, st.clean_calls, st.fired_any) == (5, 5, 0)
    assert st.sigma_sum == 5 * float(np.float32(r0.sigma_hat))
    assert np.array_equal(S.cpu().numpy(), S0) and hp.side.rebuilds == rebuilds
    # the graph reads C in place: a fault written into the same buffer is seen by the next replay
    dC[100, 200] += 0.5
    g.replay()
    g.replay()
    torch.cuda.synchronize()
    st = fpsk.read_probe_state(state)
    assert (st.calls, st.clean_calls, st.fired_any, st.first_fired_call) == (7, 5, 1, 6)
    assert fpsk.read_probe_result(res).fired == 1


def test_recalibration_from_the_accumulated_noise():
    n1 = n2 = n3 = 1024
    m = 64
    A, Bm, Cm = _case("gauss_scaled", n1, n2, n3, W.BF16, 31)
    dA, dB, dC = A.cuda(), Bm.cuda(), Cm.cuda()
    hp = fpsk.HashedProbe(n1, n2, n3, m, seed=6)
    res = fpsk.new_probe_result()
    state = fpsk.new_probe_state()
    calls = 0
    while not fpsk.recalibration_due(calls):
        hp(dA, dB, dC, res, state=state)
        calls += 1
    st = fpsk.read_probe_state(state)
    assert calls == 16 and st.calls == 16 and st.clean_calls == 16
    sigma_bar = st.sigma_sum / st.clean_calls
    rms = O.rms_c_estimate(Cm.numpy())
    got = fpsk.probe_recalibrate(n1, n3, sigma_bar, rms, m)
    assert got == O.recalibrate_probe(n1, n3, sigma_bar, rms, m)
    # the oracle's sketch at the same bucket count gives the same plan input
    ref, _ = O.probe_hashed(_f64(A), _f64(Bm), Cm.numpy(), 6, 0, m)
    assert sigma_bar == pytest.approx(ref.sigma_hat, rel=0.05)


# ---------------------------------------------------------------- weight stored transposed (C = A W^T)
@pytest.mark.parametrize("shape,m,dtype", [((512, 256, 384), 32, W.BF16), ((1024, 1032, 2048), 128, W.FP16),
                                           ((130, 72, 100), 5, W.BF16)])
def test_transposed_weight_layout(shape, m, dtype):
    n1, n2, n3 = shape
    A, Bm, Cm = _case("gauss_scaled", n1, n2, n3, dtype, 23)
    Cm[n1 // 2, n3 // 3] += 0.75
    Wt = Bm.t().contiguous()                                   # n3 x n2, what an x W^T layer holds
    ref, S_ref = O.probe_hashed(_f64(A), _f64(Wt).T, Cm.numpy(), 17, 1, m)
    h1, _ = O.hash_round(17, 1, 0, n1, m)
    h2, _ = O.hash_round(17, 1, 1, n3, m)
    denom = O.abs_sketch(O.abs_product(_f64(A), _f64(Bm)), h1, h2, m)
    hp_t = fpsk.HashedProbe(n1, n2, n3, m, seed=17, rnd=1, b_transposed=True)
    got_t, S_t = _run(hp_t, A.cuda(), Wt.cuda(), Cm.cuda())
    assert got_t.status == 0 and got_t.fired == 1 and ref.fired and got_t.argmax_col == ref.argmax_col
    assert np.all(np.abs(S_t - S_ref) <= TOL * denom + 1e-30)
    # same additions in the same order as the untransposed layout: identical bits
    hp = fpsk.HashedProbe(n1, n2, n3, m, seed=17, rnd=1)
    got, S = _run(hp, A.cuda(), Bm.cuda(), Cm.cuda())
    assert np.array_equal(S, S_t) and got.tau == got_t.tau and got.sigma_hat == got_t.sigma_hat
    # a padded leading dimension of W
    big = torch.zeros(n3, n2 + 16, dtype=Wt.dtype, device="cuda")
    big[:, :n2] = Wt.cuda()
    hp_p = fpsk.HashedProbe(n1, n2, n3, m, seed=17, rnd=1, b_transposed=True)
    got_p, S_p = _run(hp_p, A.cuda(), big[:, :n2], Cm.cuda())
    assert np.array_equal(S_p, S_t)


# ---------------------------------------------------------------- the probe as one launch
# With tensor_cores = 1, at most 256 buckets and inputs the bulk copies can address, stream, contraction, combine and
# verdict run as one cooperative kernel (P goes to the tensor cores as FP16 planes scaled per bucket and column
# segment of A).  What it returns is held to the same bars as the three-launch form.
FUSED_SHAPES = [
    # (n1, n2, n3, m)
    (1024, 4096, 1024, 256),      # two column segments of A, one item per contracting CTA
    (512, 6152, 768, 128),        # a ragged last segment, one row tile
    (384, 2048 * 20, 256, 256),   # twenty segments: more items than contracting CTAs (a CTA takes several in turn)
    (2048, 520, 1028, 200),       # buckets that do not fill the second row tile, K below one segment
]


@pytest.mark.parametrize("shape", FUSED_SHAPES)
@pytest.mark.parametrize("dtype", [W.FP16, W.BF16])
def test_one_launch_form_against_the_oracle(shape, dtype):
    n1, n2, n3, m = shape
    A, Bm, Cm = _case("gauss_scaled", n1, n2, n3, dtype, 7)
    A64, B64 = _f64(A), _f64(Bm)
    ref, S_ref = O.probe_hashed(A64, B64, Cm.numpy(), 33, 2, m)
    h1, _ = O.hash_round(33, 2, 0, n1, m)
    h2, _ = O.hash_round(33, 2, 1, n3, m)
    denom = O.abs_sketch(O.abs_product(A64, B64), h1, h2, m)
    hp = fpsk.HashedProbe(n1, n2, n3, m, seed=33, rnd=2)
    dA, dB, dC = A.cuda(), Bm.cuda(), Cm.cuda()
    pr = fpsk.default_params(tensor_cores=1)
    _run(hp, dA, dB, dC, params=pr)                                   # builds the B side
    n0 = fpsk.launch_count()
    got, S = _run(hp, dA, dB, dC, params=pr)
    assert fpsk.launch_count() - n0 == 1                              # the whole probe was one kernel
    assert got.status == 0
    assert np.all(np.abs(S - S_ref) <= TOL * denom + 1e-30)
    assert got.tau == pytest.approx(ref.tau, rel=1e-6)
    v = O.probe_verdict(S.ravel(), ref.tau, n_rows=1)
    assert got.sigma_hat == pytest.approx(v.sigma_hat, rel=1e-4, abs=1e-30)
    assert got.thr == pytest.approx(v.thr, rel=1e-4, abs=1e-30)
    assert got.max_abs == pytest.approx(v.max_abs, rel=1e-6, abs=1e-30)
    assert got.argmax_col == v.argmax_col and got.nonfinite == 0
    # bit-identical from call to call, and against the three-launch form within the rounding of the two contractions
    got2, S2 = _run(hp, dA, dB, dC, params=pr)
    assert np.array_equal(S, S2) and got2.sigma_hat == got.sigma_hat
    n0 = fpsk.launch_count()
    got3, S3 = _run(hp, dA, dB, dC, params=fpsk.default_params(tensor_cores=0))
    assert fpsk.launch_count() - n0 == 3
    assert np.all(np.abs(S3 - S) <= 2 * TOL * denom + 1e-30)
    # a fault of a few percent of rms(C) fires in both forms at the same bucket
    f = W.faults_additive(n1, n3, W.rms(Cm), 3, 1, 0.05, 0.09, "small")
    Cf, _ = W.inject(Cm, f)
    dCf = Cf.cuda()
    g1, _ = _run(hp, dA, dB, dCf, params=pr)
    g0, _ = _run(hp, dA, dB, dCf, params=fpsk.default_params(tensor_cores=0))
    want = int(h1[f[0].i]) * m + int(h2[f[0].j])
    assert g1.fired == 1 and g0.fired == 1 and g1.argmax_col == g0.argmax_col == want


def test_one_launch_form_integer_products_and_nonfinite():
    n1, n2, n3, m = 768, 4104, 512, 256
    A, Bm = W.operands("integer", n1, n2, n3, W.FP16, 9)
    Cm = W.cpu_fp32_product(A, Bm)
    Cm[5, 7] += 4.0
    ref, S_ref = O.probe_hashed(_f64(A), _f64(Bm), Cm.numpy(), 2, 0, m)
    hp = fpsk.HashedProbe(n1, n2, n3, m, seed=2)
    pr = fpsk.default_params(tensor_cores=1)
    dA, dB = A.cuda(), Bm.cuda()
    got, S = _run(hp, dA, dB, Cm.cuda(), params=pr)
    assert np.array_equal(S, S_ref)                                   # integers survive the split into two FP16 terms exactly
    assert got.fired == 1 and got.argmax_col == ref.argmax_col and got.max_abs == ref.max_abs
    for bad in (float("nan"), float("inf")):
        Cb = Cm.clone()
        Cb[100, 100] = bad
        got, _ = _run(hp, dA, dB, Cb.cuda(), params=pr)
        assert got.status == 0 and got.fired == 1 and got.nonfinite == 1
    Ab = A.clone()
    Ab[17, 2050] = float("inf")                                       # a non-finite operand: its bucket's planes carry it
    got, _ = _run(hp, Ab.cuda(), dB, Cm.cuda(), params=pr)
    assert got.status == 0 and got.fired == 1 and got.nonfinite == 1


def test_one_launch_form_replays_from_a_cuda_graph():
    n1, n2, n3, m = 1024, 4096, 1024, 256
    A, Bm, Cm = _case("gauss_scaled", n1, n2, n3, W.BF16, 23)
    dA, dB, dC = A.cuda(), Bm.cuda(), Cm.cuda().clone()
    hp = fpsk.HashedProbe(n1, n2, n3, m, seed=4)
    pr = fpsk.default_params(tensor_cores=1)
    res = fpsk.new_probe_result()
    state = fpsk.new_probe_state()
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        hp(dA, dB, dC, res, params=pr)
    side.synchronize()
    r0 = fpsk.read_probe_result(res)
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        hp(dA, dB, dC, res, params=pr, state=state)
    for _ in range(4):
        g.replay()
    torch.cuda.synchronize()
    st = fpsk.read_probe_state(state)
    assert (st.calls, st.clean_calls, st.fired_any) == (4, 4, 0)
    assert st.sigma_sum == 4 * float(np.float32(r0.sigma_hat))
    dC[10, 20] += 0.5
    g.replay()
    torch.cuda.synchronize()
    st = fpsk.read_probe_state(state)
    assert (st.calls, st.fired_any, st.first_fired_call) == (5, 1, 5)


@pytest.mark.parametrize("shape", [(100, 512, 64, 256), (40, 8, 8, 256), (4096, 16, 4096, 200), (2056, 6152, 1028, 129)])
def test_one_launch_form_sparse_buckets_and_short_inner_dimensions(shape):
    """More buckets than rows or columns (most buckets empty), an inner dimension below one K block, a bucket count
    that fills neither row tile: S, tau and the verdict still follow the oracle's."""
    n1, n2, n3, m = shape
    A, Bm = W.operands("gauss_scaled", n1, n2, n3, W.BF16, 3)
    Cm = W.cpu_fp32_product(A, Bm)
    A64, B64 = _f64(A), _f64(Bm)
    ref, S_ref = O.probe_hashed(A64, B64, Cm.numpy(), 5, 1, m)
    h1, _ = O.hash_round(5, 1, 0, n1, m)
    h2, _ = O.hash_round(5, 1, 1, n3, m)
    denom = O.abs_sketch(O.abs_product(A64, B64), h1, h2, m)
    hp = fpsk.HashedProbe(n1, n2, n3, m, seed=5, rnd=1)
    pr = fpsk.default_params(tensor_cores=1)
    dA, dB, dC = A.cuda(), Bm.cuda(), Cm.cuda()
    _run(hp, dA, dB, dC, params=pr)
    n0 = fpsk.launch_count()
    got, S = _run(hp, dA, dB, dC, params=pr)
    assert fpsk.launch_count() - n0 == 1 and got.status == 0
    assert np.all(np.abs(S - S_ref) <= TOL * denom + 1e-30)
    assert got.tau == pytest.approx(ref.tau, rel=1e-6)
    v = O.probe_verdict(S.ravel(), ref.tau, n_rows=1)
    assert got.sigma_hat == pytest.approx(v.sigma_hat, rel=1e-4, abs=1e-30)
    assert got.argmax_col == v.argmax_col and got.nonfinite == 0
    if abs(v.max_abs - v.thr) > 1e-3 * v.thr:
        assert bool(got.fired) == v.fired
