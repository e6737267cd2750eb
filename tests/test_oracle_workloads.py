"""The oracle on floating-point products shaped like the benchmark's small case: a clean
product stays clean, each injected fault comes back with its exact coordinate and with the
magnitude that was written, and nothing else is ever reported."""
import numpy as np
import pytest

import oracle as O
from paper_2609_19758_b200 import workloads as W


def _case(seed, n=256, dtype=W.FP16, kind="uniform"):
    A, B = W.operands(kind, n, n, n, dtype, seed)
    C = W.cpu_fp32_product(A, B)
    return A, B, C


def test_small_square_fp16_clean_and_single_faults():
    A, B, C = _case(1)
    A64, B64 = A.double().numpy(), B.double().numpy()
    p = O.Params(s_budget=1, delta_max=1)
    nz = O.measure_noise(A64, B64, C.numpy(), seed=7, dtype=O.FP16, params=p)
    assert nz.m0 == 16 and 16 <= nz.m_loc <= 64 and 0 <= nz.radius <= 16
    assert 0.02 < nz.c_hat < 1.0            # same order as the paper's normalized constant
    tau = O.analytic_tau(A64, B64, 256)
    E = O.error_matrix(A64, B64, C.numpy())
    assert not O.probe_verdict(O.probe_sketch(E), tau, n_rows=256).fired
    p.radius = nz.radius
    assert O.localize(A64, B64, C.numpy(), 7, nz.m_loc, O.FP16, p, E=E) == []
    rms = W.rms(C)
    for s in (1, 2, 3):
        f = W.faults_additive(256, 256, rms, s, 1, 0.5, 0.5, "typical")
        Cf, changes = W.inject(C, f)
        Ef = O.error_matrix(A64, B64, Cf.numpy())
        v = O.probe_verdict(O.probe_sketch(Ef), tau, n_rows=256)
        assert v.fired and v.argmax_col == f[0].j
        F = O.localize(A64, B64, Cf.numpy(), 7, nz.m_loc, O.FP16, p, E=Ef)
        assert [(x.i, x.j) for x in F] == [(f[0].i, f[0].j)]
        # reported delta = gamma - C_ij = E_ij = -(change) up to the GEMM's own FP32 rounding
        assert F[0].delta == pytest.approx(-changes[0], abs=2e-5)
        assert abs(changes[0]) == pytest.approx(0.5 * rms, rel=1e-3)


def test_bf16_multi_fault_small_magnitudes():
    n = 512
    A, B = W.operands("gauss_scaled", n, n, n, W.BF16, 3)
    C = W.cpu_fp32_product(A, B)
    A64, B64 = A.double().numpy(), B.double().numpy()
    rms = W.rms(C)
    assert rms == pytest.approx(1.0, rel=0.05)
    p = O.Params(s_budget=4)
    nz = O.measure_noise(A64, B64, C.numpy(), seed=11, dtype=O.BF16, params=p)
    p.radius = nz.radius
    f = W.faults_additive(n, n, rms, 5, 4, 0.02, 0.09, "small")
    Cf, changes = W.inject(C, f)
    F = O.localize(A64, B64, Cf.numpy(), 11, nz.m_loc, O.BF16, p)
    assert {(x.i, x.j) for x in F} == {(x.i, x.j) for x in f}
    want = {(x.i, x.j): -c for x, c in zip(f, changes)}
    for x in F:
        assert x.delta == pytest.approx(want[(x.i, x.j)], abs=1e-5)


def test_injector_shapes():
    C = W.cpu_fp32_product(*W.operands("uniform", 64, 64, 64, W.FP16, 9))
    fl = W.faults_mixed16(C, W.rms(C), 4)
    assert len(fl) == 16 and len({(f.i, f.j) for f in fl}) == 16
    rows = [f.i for f in fl]
    cols = [f.j for f in fl]
    assert max(rows.count(r) for r in rows) >= 4 and max(cols.count(c) for c in cols) >= 3
    Cf, ch = W.inject(C, fl)
    assert all(abs(c) >= 0.0199 * W.rms(C) for c in ch)
    assert int((Cf != C).sum()) == 16
    # an exponent-flip fault multiplies the stored entry by a power of two
    for f in fl:
        if f.kind == "scale":
            assert float(Cf[f.i, f.j]) == float(C[f.i, f.j]) * 2.0 ** f.value
