"""The split-FP16 tensor-core contraction (tcgen05) behind `tensor_cores = 1`: same results as the FP32
FMA contraction within the 1e-5 tolerance, bit-exact on integer products, and a measured sketch noise
that is not above the FMA path's (the gate for using it; Section "Implementation" warns that a
single-pass reduced-precision product raised the floor 419x).  The bucket sums are scaled by a power of
two into FP16 range before they are split, so operands of any magnitude must behave the same."""
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
    return A, Bm, harness.vendor_gemm_fp32(A.cuda(), Bm.cuda()).cpu()


@pytest.mark.parametrize("shape,m_b,dtype", [((1024, 1024, 1024), 384, W.BF16), ((1536, 520, 1280), 400, W.FP16),
                                             ((2048, 2048, 2048), 512, W.BF16)])
def test_localize_agrees_with_the_oracle_and_with_the_fma_path(shape, m_b, dtype):
    n1, n2, n3 = shape
    A, Bm, Cm = _case("gauss_scaled", n1, n2, n3, dtype, 5)
    rms = W.rms(Cm)
    faults = W.faults_additive(n1, n3, rms, 3, 4, 0.03, 0.09, "small")
    Cf, ch = W.inject(Cm, faults)
    dA, dB, dF = A.cuda(), Bm.cuda(), Cf.cuda()
    A64, B64 = _f64(A), _f64(Bm)
    ref = O.localize(A64, B64, Cf.numpy(), 77, m_b, dtype, O.Params(s_budget=4, radius=4))
    rset = {(f.i, f.j) for f in ref}
    rmap = {(f.i, f.j): f for f in ref}
    results = {}
    for tc in (0, 1):
        p = fpsk.default_params(s_budget=4, radius=4, tensor_cores=tc)
        ws = fpsk.workspace(n1, n2, n3, m_b, p)
        got = fpsk.localize(dA, dB, dF, 77, m_b, ws, p)
        results[tc] = got
        assert {(f.i, f.j) for f in got} == rset == {(f.i, f.j) for f in faults}
        for f in got:
            a = np.abs(A64[f.i, :]) @ np.abs(B64[:, f.j])
            assert abs(f.delta - rmap[(f.i, f.j)].delta) <= TOL * a
    assert [(f.i, f.j, f.delta, f.round) for f in results[0]] == [(f.i, f.j, f.delta, f.round) for f in results[1]]


def test_integer_products_localize_exactly():
    n1, n2, n3, m_b = 768, 256, 640, 384
    A, Bm = W.operands("integer", n1, n2, n3, W.FP16, 31, lim=8)
    Cm = W.cpu_fp32_product(A, Bm)
    coords = [(5, 1), (5, 9), (300, 630), (767, 639), (0, 0), (412, 77)]
    faults = [W.InjectedFault(i, j, "add", 3.0 + t, "typical") for t, (i, j) in enumerate(coords)]
    Cf, ch = W.inject(Cm, faults)
    p = fpsk.default_params(radius=1, rounds=3, tensor_cores=1)
    ws = fpsk.workspace(n1, n2, n3, m_b, p)
    got = fpsk.localize(A.cuda(), Bm.cuda(), Cf.cuda(), 2024, m_b, ws, p)
    assert {(f.i, f.j) for f in got} == set(coords)
    for f in got:
        assert f.delta == -(3.0 + coords.index((f.i, f.j)))


@pytest.mark.parametrize("n,dtype", [(2048, W.BF16), (2048, W.FP16)])
def test_measured_noise_is_not_above_the_fma_path(n, dtype):
    A, Bm, Cm = _case("gauss_scaled", n, n, n, dtype, 9)
    dA, dB, dC = A.cuda(), Bm.cuda(), Cm.cuda()
    sig = {}
    for tc in (0, 1):
        p = fpsk.default_params(tensor_cores=tc)
        ws = fpsk.workspace(n, n, n, 512, p)
        sig[tc] = fpsk.measure_noise(dA, dB, dC, 5, ws, 512, p)
    # what an exact verifier would see: the GEMM's own rounding, sketched in FP64
    h1, v1 = O.hash_round(5, 0, 0, n, 512)
    h2, v2 = O.hash_round(5, 0, 1, n, 512)
    E = _f64(A) @ _f64(Bm) - Cm.numpy().astype(np.float64)
    ref = O.sigma_clip(O.hashed_sum_sketch(E, h1, v1, h2, v2, 512))
    assert sig[1].sigma_clip <= 1.02 * sig[0].sigma_clip
    # It may even fall below the exact verifier's: the product under test comes from the same tensor cores, and
    # the part of its rounding that is systematic (accumulation that is not round-to-nearest) is reproduced by
    # the verifier's own contraction and cancels in the sketch.
    assert 0.5 * ref <= sig[1].sigma_clip <= 1.5 * ref
    assert sig[0].rms_c == sig[1].rms_c


def test_small_bucket_counts_keep_the_fma_contraction():
    """Below the crossover the flag changes nothing (same kernels, same bits)."""
    n, m_b = 512, 128
    A, Bm, Cm = _case("gauss_scaled", n, n, n, W.BF16, 17)
    dA, dB, dC = A.cuda(), Bm.cuda(), Cm.cuda()
    out = []
    for tc in (0, 1):
        p = fpsk.default_params(tensor_cores=tc)
        ws = fpsk.workspace(n, n, n, m_b, p)
        out.append(fpsk.measure_noise(dA, dB, dC, 5, ws, m_b, p))
    assert out[0].sigma_clip == out[1].sigma_clip and out[0].sigma_mad == out[1].sigma_mad


@pytest.mark.parametrize("log2_scale_a,log2_scale_b", [(40, 0), (-40, 0), (60, -60), (-30, -30), (100, 10)])
def test_operand_magnitude_does_not_matter(log2_scale_a, log2_scale_b):
    """Powers of two on A and B only move exponents: the same faults are found, with deltas scaled exactly."""
    n1, n2, n3, m_b = 1024, 768, 1280, 400
    A, Bm = W.operands("gauss_scaled", n1, n2, n3, W.BF16, 12)
    base = None
    for sa, sb in ((0, 0), (log2_scale_a, log2_scale_b)):
        As = (A.double() * 2.0 ** sa).to(torch.bfloat16)
        Bs = (Bm.double() * 2.0 ** sb).to(torch.bfloat16)
        Cm = harness.vendor_gemm_fp32(As.cuda(), Bs.cuda()).cpu()
        faults = W.faults_additive(n1, n3, W.rms(Cm), 3, 4, 0.05, 0.09, "small")
        Cf, _ = W.inject(Cm, faults)
        p = fpsk.default_params(s_budget=4, radius=4, tensor_cores=1)
        ws = fpsk.workspace(n1, n2, n3, m_b, p)
        got = fpsk.localize(As.cuda(), Bs.cuda(), Cf.cuda(), 77, m_b, ws, p)
        nz = fpsk.measure_noise(As.cuda(), Bs.cuda(), Cm.cuda(), 5, ws, m_b, p)
        assert {(f.i, f.j) for f in got} == {(f.i, f.j) for f in faults}
        rec = (sorted((f.i, f.j, f.delta * 2.0 ** -(sa + sb)) for f in got), nz.sigma_clip * 2.0 ** -(sa + sb))
        if base is None:
            base = rec
        else:
            # scaling by powers of two is exact in every step of the verifier (no over- or underflow here)
            assert [(i, j) for i, j, _ in rec[0]] == [(i, j) for i, j, _ in base[0]]
            for (_, _, d), (_, _, d0) in zip(rec[0], base[0]):
                assert d == pytest.approx(d0, rel=1e-6)
            assert rec[1] == pytest.approx(base[1], rel=1e-3)


def test_all_zero_and_huge_operands_do_not_break_the_scaling():
    n, m_b = 512, 384
    A = torch.zeros(n, n, dtype=torch.bfloat16)
    Bm = torch.zeros(n, n, dtype=torch.bfloat16)
    Cm = torch.zeros(n, n, dtype=torch.float32)
    p = fpsk.default_params(tensor_cores=1, radius=2)
    ws = fpsk.workspace(n, n, n, m_b, p)
    assert fpsk.localize(A.cuda(), Bm.cuda(), Cm.cuda(), 1, m_b, ws, p) == []
    # the largest finite BF16 in A: the bound (largest bucket) x max|A| overflows FP32 -> scale 1, sums may overflow
    # FP16 planes; the call must still return (nonfinite sketches select nothing that confirms)
    A2, B2 = W.operands("gauss_scaled", n, n, n, W.BF16, 4)
    A2[3, 5] = torch.finfo(torch.bfloat16).max
    C2 = harness.vendor_gemm_fp32(A2.cuda(), B2.cuda())
    got = fpsk.localize(A2.cuda(), B2.cuda(), C2, 1, m_b, ws, p)
    assert isinstance(got, list)


@pytest.mark.parametrize("tc", [0, 1])
def test_more_keys_than_one_pass_of_the_select_kernel_holds(tc):
    """1200^2 = 1.44 M buckets: the radix selects take their keys in more than one batch per digit."""
    n1, n2, n3, m_b = 4800, 128, 4800, 1200
    A, Bm = W.operands("gauss_scaled", n1, n2, n3, W.BF16, 8)
    Cm = harness.vendor_gemm_fp32(A.cuda(), Bm.cuda()).cpu()
    faults = W.faults_additive(n1, n3, W.rms(Cm), 6, 5, 0.05, 0.09, "small")
    Cf, _ = W.inject(Cm, faults)
    A64, B64 = _f64(A), _f64(Bm)
    ref = O.localize(A64, B64, Cf.numpy(), 31, m_b, W.BF16, O.Params(s_budget=5, radius=3))
    rmap = {(f.i, f.j): f.delta for f in ref}
    p = fpsk.default_params(s_budget=5, radius=3, tensor_cores=tc)
    ws = fpsk.workspace(n1, n2, n3, m_b, p)
    got = fpsk.localize(A.cuda(), Bm.cuda(), Cf.cuda(), 31, m_b, ws, p)
    assert {(f.i, f.j) for f in got} == set(rmap) == {(f.i, f.j) for f in faults}
    for f in got:
        a = np.abs(A64[f.i, :]) @ np.abs(B64[:, f.j])
        assert abs(f.delta - rmap[(f.i, f.j)]) <= TOL * a
    if tc == 0:
        # the estimates against the definitions applied to the very sketch they were taken from (FP32, as the kernels
        # compute them): lower medians by exact selection, so equality is bit for bit
        S, _, _ = fpsk.sketches(A.cuda(), Bm.cuda(), Cm.cuda(), 5, 0, m_b, ws, moments=False)
        a = np.abs(S.cpu().numpy().ravel())
        rank = (a.size - 1) // 2
        med = np.partition(a, rank)[rank]
        dev = np.abs(a - med)
        mad = np.float32(1.4826) * np.partition(dev, rank)[rank]
        mean = np.float32(a.astype(np.float64).sum() / a.size)
        nz = fpsk.measure_noise(A.cuda(), Bm.cuda(), Cm.cuda(), 5, ws, m_b, p)
        assert np.float32(nz.sigma_mad) == mad
        clip = np.float32(1.2533) * np.float32(np.minimum(a, np.float32(5) * mean).astype(np.float64).sum() / a.size)
        assert nz.sigma_clip == pytest.approx(float(clip), rel=1e-5)


@pytest.mark.parametrize("m_b,mad_of_abs", [(300, 1), (300, 0), (1024, 1), (1024, 0), (17, 1)])
def test_sigma_mad_is_the_exact_selection_on_the_sketch(m_b, mad_of_abs):
    """sigma_MAD of `fpsk_measure_noise` = 1.4826 x lower median of the deviations from the lower median, bit for
    bit, on the sketch the same kernels produce (FMA contraction, so that `fpsk_sketches` gives that sketch)."""
    n = 1536
    A, Bm = W.operands("gauss_scaled", n, n, n, W.FP16, 41)
    dA, dB = A.cuda(), Bm.cuda()
    dC = harness.vendor_gemm_fp32(dA, dB)
    p = fpsk.default_params(tensor_cores=0, mad_of_abs=mad_of_abs)
    ws = fpsk.workspace(n, n, n, m_b, p)
    S, _, _ = fpsk.sketches(dA, dB, dC, 9, 0, m_b, ws, moments=False)
    x = S.cpu().numpy().ravel()
    a = np.abs(x) if mad_of_abs else x
    rank = (a.size - 1) // 2
    med = np.partition(a, rank)[rank]
    dev = np.abs(a - med)
    mad = np.float32(1.4826) * np.partition(dev, rank)[rank]
    nz = fpsk.measure_noise(dA, dB, dC, 9, ws, m_b, p)
    assert np.float32(nz.sigma_mad) == mad


# ------------------------------------------------------------------ the sketch builder itself, element by element
def _sketch_refs(A, Bm, Cm, seed, rnd, m_b):
    n1, n3 = A.shape[0], Bm.shape[1]
    A64, B64 = _f64(A), _f64(Bm)
    E = O.error_matrix(A64, B64, Cm.numpy())
    h1, v1 = O.hash_round(seed, rnd, 0, n1, m_b)
    h2, v2 = O.hash_round(seed, rnd, 1, n3, m_b)
    return O.moment_sketches(E, h1, v1, h2, v2, m_b), O.abs_sketch(O.abs_product(A64, B64), h1, h2, m_b)


@pytest.mark.parametrize("shape,m_b,dtype", [((1024, 1024, 1024), 384, W.BF16), ((1536, 520, 1280), 400, W.FP16),
                                             ((2048, 1032, 4096), 1024, W.BF16), ((4096, 512, 2048), 1024, W.FP16)])
@pytest.mark.parametrize("b_transposed", [0, 1])
def test_tensor_core_sketches_element_by_element(shape, m_b, dtype, b_transposed):
    """S, R and T of the tcgen05 sketch builder (planes written by the compressions, split-K partials, combine)
    against the oracle's definition, every bucket, for B as k x n and as the weight W = B^T."""
    n1, n2, n3 = shape
    A, Bm, Cm = _case("uniform" if dtype == W.FP16 else "gauss_scaled", n1, n2, n3, dtype, 19)
    Cf, _ = W.inject(Cm, W.faults_additive(n1, n3, W.rms(Cm), 3, 4, 0.02, 1.0, "small"))
    (So, Ro, To), ABS = _sketch_refs(A, Bm, Cf, 2024, 1, m_b)
    p = fpsk.default_params(tensor_cores=1, b_transposed=b_transposed)
    ws = fpsk.workspace(n1, n2, n3, m_b, p)
    dB = Bm.t().contiguous().cuda() if b_transposed else Bm.cuda()
    S, R, T = fpsk.sketches(A.cuda(), dB, Cf.cuda(), 2024, 1, m_b, ws, params=p)
    S2, _, _ = fpsk.sketches(A.cuda(), dB, Cf.cuda(), 2024, 1, m_b, ws, moments=False, params=p)
    torch.cuda.synchronize()
    for g, o in ((S, So), (R, Ro), (T, To), (S2, So)):
        assert np.all(np.abs(g.cpu().numpy().astype(np.float64) - o) <= TOL * ABS + 1e-30)


@pytest.mark.parametrize("b_transposed", [0, 1])
def test_tensor_core_sketches_are_bit_exact_on_integer_products(b_transposed):
    n1, n2, n3, m_b = 768, 264, 640, 384
    A, Bm = W.operands("integer", n1, n2, n3, W.FP16, 31, lim=8)
    Cm = W.cpu_fp32_product(A, Bm)
    Cm[5, 1] += 3.0
    Cm[767, 639] -= 7.0
    Cm[300, 630] += 1.0
    (So, Ro, To), _ = _sketch_refs(A, Bm, Cm, 77, 2, m_b)
    p = fpsk.default_params(tensor_cores=1, b_transposed=b_transposed)
    ws = fpsk.workspace(n1, n2, n3, m_b, p)
    dB = Bm.t().contiguous().cuda() if b_transposed else Bm.cuda()
    S, R, T = fpsk.sketches(A.cuda(), dB, Cm.cuda(), 77, 2, m_b, ws, params=p)
    for g, o in ((S, So), (R, Ro), (T, To)):
        assert np.array_equal(g.cpu().numpy().astype(np.float64), o)


# ------------------------------------------------------------------ Eq. (recover) with no window to hide behind
@pytest.mark.parametrize("shape,m_b,tc", [((64, 16, 48), 16, 0), ((300, 40, 520), 64, 0), ((768, 256, 640), 384, 0),
                                          ((768, 256, 640), 384, 1), ((1000, 72, 1536), 512, 1)])
@pytest.mark.parametrize("n_faults", [1, 5])
def test_radius_zero_decodes_the_exact_coordinate(shape, m_b, tc, n_faults):
    """Exact integer products, radius 0: the only entry ever recomputed for a bucket is the one Eq. (recover)
    names, so the moments at the kept buckets and the decode must be right to the unit.  The fault list must be
    the oracle's: coordinates, round, bucket and exact magnitude (faults that collide in every round are missed
    by both)."""
    n1, n2, n3 = shape
    A, Bm = W.operands("integer", n1, n2, n3, W.FP16, 31, lim=8)
    Cm = W.cpu_fp32_product(A, Bm)
    g = np.random.default_rng(n1 + n_faults)
    coords = [(n1 - 1, n3 - 1)] if n_faults == 1 else []
    while len(coords) < n_faults:
        c = (int(g.integers(n1)), int(g.integers(n3)))
        if c not in coords:
            coords.append(c)
    faults = [W.InjectedFault(i, j, "add", float((t + 2) * (1 if t % 2 else -1)), "typical") for t, (i, j) in enumerate(coords)]
    Cf, _ = W.inject(Cm, faults)
    p = fpsk.default_params(radius=0, tensor_cores=tc)
    ws = fpsk.workspace(n1, n2, n3, m_b, p)
    got = fpsk.localize(A.cuda(), Bm.cuda(), Cf.cuda(), 4242, m_b, ws, p)
    ref = O.localize(_f64(A), _f64(Bm), Cf.numpy(), 4242, m_b, W.FP16, O.Params(radius=0))
    assert [(f.i, f.j, f.delta, f.round, f.bucket_a, f.bucket_b) for f in got] == \
           [(f.i, f.j, f.delta, f.round, f.bucket_a, f.bucket_b) for f in ref]
    assert {(f.i, f.j) for f in got} == set(coords)
    for f in got:
        assert f.delta == -faults[coords.index((f.i, f.j))].value
