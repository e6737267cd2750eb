"""Algorithm 2 complete on the GPU (probe, exact scan, absolute repairs, localization, apply,
second probe) against the oracle: same coordinates, same absolute / relative split, repaired
values within tolerance, the product restored."""
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


def _int(n1, n2, n3, seed):
    A, Bm = W.operands("integer", n1, n2, n3, W.FP16, seed, lim=8)
    return A, Bm, W.cpu_fp32_product(A, Bm)


def test_exact_integer_product_with_nonfinite_entries_is_restored_bit_for_bit():
    A, Bm, C0 = _int(32, 8, 32, 7)
    C = C0.clone()
    C[5, 3] = float("nan")
    C[5, 20] += 6.0
    C[11, 9] = float("inf")
    C[30, 9] -= 4.0
    C[17, 17] = -float(np.float32(O.FP32_MAX / 4))
    C[2, 2] += 3.0
    p = fpsk.default_params(radius=1, rounds=6)
    po = O.Params(radius=1, rounds=6)
    dA, dB, dC = A.cuda(), Bm.cuda(), C.cuda()
    ws = fpsk.repair_workspace(32, 8, 32, 6, p)
    got, rep = fpsk.verify_repair(dA, dB, dC, 2024, ws, 6, p)
    out_o, F_o, rep_o = O.verify_repair(A.double().numpy(), Bm.double().numpy(), C.numpy(), 2024, O.FP16, po, m_b=6)
    assert rep.state == rep_o["state"] == 1 and rep.n_absolute == rep_o["n_absolute"] == 3
    assert rep.first_probe.fired == 1 and rep.first_probe.nonfinite == 1 and rep.second_probe.fired == 0
    assert [(f.i, f.j, f.round < 0, f.delta) for f in got] == [(f.i, f.j, f.round < 0, f.delta) for f in F_o]
    assert torch.equal(dC.cpu(), C0)
    assert np.array_equal(out_o, C0.numpy())


def test_clean_product_is_untouched_and_only_the_probe_runs():
    n = 512
    A, Bm = W.operands("gauss_scaled", n, n, n, W.BF16, 3)
    dA, dB = A.cuda(), Bm.cuda()
    dC = harness.vendor_gemm_fp32(dA, dB)
    keep = dC.clone()
    ws = fpsk.repair_workspace(n, n, n, 0)
    before = fpsk.launch_count()
    got, rep = fpsk.verify_repair(dA, dB, dC, 5, ws)
    assert rep.state == 0 and got == [] and torch.equal(dC, keep)
    assert fpsk.launch_count() - before == 1


@pytest.mark.parametrize("n,dtype,kind", [(1024, W.BF16, "gauss_scaled"), (768, W.FP16, "uniform")])
def test_mixed_faults_are_repaired_and_match_the_oracle(n, dtype, kind):
    A, Bm = W.operands(kind, n, n, n, dtype, 9)
    dA, dB = A.cuda(), Bm.cuda()
    dC = harness.vendor_gemm_fp32(dA, dB)
    clean = dC.clone()
    rms = float(torch.sqrt(torch.mean(dC.double() ** 2)))
    faults = W.faults_additive(n, n, rms, 4, 4, 0.05, 0.5, "small")
    for f in faults:
        dC[f.i, f.j] += f.value
    dC[7, 7] = float("nan")
    dC[7, 100] = float("inf")
    dC[300, 7] = 1e38
    bad = dC.clone()
    p = fpsk.default_params(s_budget=8)
    po = O.Params(s_budget=8)
    ws = fpsk.repair_workspace(n, n, n, 0, p)
    got, rep = fpsk.verify_repair(dA, dB, dC, 11, ws, 0, p)
    A64, B64 = A.double().numpy(), Bm.double().numpy()
    out_o, F_o, rep_o = O.verify_repair(A64, B64, bad.cpu().numpy(), 11, dtype, po)
    want = {(f.i, f.j) for f in faults} | {(7, 7), (7, 100), (300, 7)}
    assert {(f.i, f.j) for f in got} == {(f.i, f.j) for f in F_o} == want
    assert rep.state == rep_o["state"] == 1 and rep.n_absolute == 3
    assert (rep.m_loc, rep.radius) == (rep_o["m_loc"], rep_o["radius"])
    omap = {(f.i, f.j): f for f in F_o}
    out = dC.cpu()
    changed = (out != bad.cpu()) & ~(torch.isnan(out) & torch.isnan(bad.cpu()))
    assert int(changed.sum()) == len(want)                       # only the reported entries were written
    for f in got:
        absab = float(np.abs(A64[f.i, :]) @ np.abs(B64[:, f.j]))
        o = omap[(f.i, f.j)]
        assert (f.round < 0) == (o.round < 0)
        assert abs(f.recompute - o.recompute) <= TOL * absab
        # the repaired entry is the fresh recomputation, i.e. the clean GEMM value up to its own rounding
        assert abs(float(out[f.i, f.j]) - float(clean[f.i, f.j])) <= 100 * 2.0 ** -23 * absab
        assert abs(float(out[f.i, f.j]) - float(out_o[f.i, f.j])) <= TOL * absab
    assert rep.second_probe.fired == 0


def test_apply_corrections_alone():
    C = torch.tensor([[1.0, 2.0, 3.0], [4.0, float("nan"), 6.0]], device="cuda")
    fl = [fpsk.Fault(0, 1, 0.5, 2.5, 2.0, 0, 0, 0), fpsk.Fault(1, 1, 7.0, 7.0, float("nan"), -1, -1, -1)]
    ws = torch.empty(1 << 20, dtype=torch.uint8, device="cuda")
    fpsk.apply_corrections(C, fl, ws)
    assert torch.equal(C.cpu(), torch.tensor([[1.0, 2.5, 3.0], [4.0, 7.0, 6.0]]))
    with pytest.raises(fpsk.FpskError) as e:
        fpsk.apply_corrections(C, [fpsk.Fault(5, 0, 1.0, 1.0, 0.0, 0, 0, 0)], ws)
    assert e.value.status == fpsk.ERR_SHAPE


def test_full_size_repair_4096_bf16():
    n = 4096
    A, Bm = W.operands("gauss_scaled", n, n, n, W.BF16, 1)
    dA, dB = A.cuda(), Bm.cuda()
    dC = harness.vendor_gemm_fp32(dA, dB)
    clean = dC.clone()
    rms = float(torch.sqrt(torch.mean(dC.double() ** 2)))
    faults = W.faults_additive(n, n, rms, 1, 4, 0.02, 0.09, "small")
    for f in faults:
        dC[f.i, f.j] += f.value
    dC[1000, 2000] = float("nan")
    p = fpsk.default_params(s_budget=4)
    ws = fpsk.repair_workspace(n, n, n, 0, p)
    got, rep = fpsk.verify_repair(dA, dB, dC, 21, ws, 0, p)
    assert rep.state == 1 and rep.n_absolute == 1
    assert {(f.i, f.j) for f in got} == {(f.i, f.j) for f in faults} | {(1000, 2000)}
    diff = (dC - clean).abs()
    assert float(diff.max()) < 1e-4          # every entry is back at its clean value up to GEMM rounding
