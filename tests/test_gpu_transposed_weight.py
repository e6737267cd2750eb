"""The x W^T layout (params.b_transposed = 1): noise measurement and localization given the weight
W = B^T (n x k, row-major) return what they return for B (k x n), bit for bit -- the B-side fold adds the
same terms in the same order, only the addressing differs -- and agree with the oracle."""
import numpy as np
import pytest
import torch

import oracle as O
from paper_2609_19758_b200 import build as B
from paper_2609_19758_b200 import fpsk, harness, workloads as W

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _lib():
    B.build()
    fpsk.lib()


def _noise_fields(nz):
    return [getattr(nz, name) for name, _ in fpsk.Noise._fields_]


@pytest.mark.parametrize("tc", [0, 1])
@pytest.mark.parametrize("shape,m_b,dtype,pad", [
    ((1024, 1024, 1024), 384, W.BF16, 0),      # tensor-core planes emitted by the fold itself
    ((700, 523, 1100), 400, W.FP16, 0),        # k not a multiple of 8: element loads, ragged planes
    ((512, 640, 2304), 96, W.BF16, 24),        # leading dimension above k, FMA contraction at either flag
    ((640, 264, 20000), 416, W.FP16, 8),       # B too wide for the eight-row staging of the k x n layout
])
def test_weight_layout_gives_the_same_bits(shape, m_b, dtype, pad, tc):
    n1, n2, n3 = shape
    A, Bm = W.operands("gauss_scaled", n1, n2, n3, dtype, 21)
    dA, dB = A.cuda(), Bm.cuda()
    Cm = harness.vendor_gemm_fp32(dA, dB).cpu()
    faults = W.faults_additive(n1, n3, W.rms(Cm), 4, 4, 0.5, 1.0, "typical")
    Cf, _ = W.inject(Cm, faults)
    dC, dF = Cm.cuda(), Cf.cuda()
    store = torch.zeros(n3, n2 + pad, dtype=dB.dtype, device="cuda")
    store[:, :n2] = dB.t()
    dW = store[:, :n2]
    assert dW.stride(0) == n2 + pad
    out = {}
    for bt, Bop in ((0, dB), (1, dW)):
        p = fpsk.default_params(s_budget=4, radius=3, tensor_cores=tc, b_transposed=bt)
        ws = fpsk.workspace(n1, n2, n3, m_b, p)
        nz = fpsk.measure_noise(dA, Bop, dC, 5, ws, m_b, p)
        got = fpsk.localize(dA, Bop, dF, 77, m_b, ws, p)
        out[bt] = (_noise_fields(nz), [(f.i, f.j, f.delta, f.round, f.bucket_a, f.bucket_b) for f in got])
    assert out[0][0] == out[1][0]
    assert out[0][1] == out[1][1]
    assert {(i, j) for (i, j, *_r) in out[1][1]} == {(f.i, f.j) for f in faults}


def test_weight_layout_agrees_with_the_oracle():
    n1, n2, n3, m_b = 768, 512, 896, 384
    A, Bm = W.operands("gauss_scaled", n1, n2, n3, W.BF16, 3)
    dA, dB = A.cuda(), Bm.cuda()
    Cm = harness.vendor_gemm_fp32(dA, dB).cpu()
    faults = W.faults_additive(n1, n3, W.rms(Cm), 9, 5, 0.03, 0.09, "small")
    Cf, _ = W.inject(Cm, faults)
    A64, B64 = A.double().numpy(), Bm.double().numpy()
    ref = O.localize(A64, B64, Cf.numpy(), 11, m_b, W.BF16, O.Params(s_budget=5, radius=4))
    rmap = {(f.i, f.j): f.delta for f in ref}
    dW = dB.t().contiguous()
    for tc in (0, 1):
        p = fpsk.default_params(s_budget=5, radius=4, tensor_cores=tc, b_transposed=1)
        ws = fpsk.workspace(n1, n2, n3, m_b, p)
        got = fpsk.localize(dA, dW, Cf.cuda(), 11, m_b, ws, p)
        assert {(f.i, f.j) for f in got} == set(rmap) == {(f.i, f.j) for f in faults}
        for f in got:
            a = np.abs(A64[f.i, :]) @ np.abs(B64[:, f.j])
            assert abs(f.delta - rmap[(f.i, f.j)]) <= 1e-5 * a


def test_entry_points_that_read_b_as_k_by_n_refuse_the_flag():
    n = 256
    A, Bm = W.operands("uniform", n, n, n, W.FP16, 1)
    dA, dB = A.cuda(), Bm.cuda()
    dC = harness.vendor_gemm_fp32(dA, dB)
    p = fpsk.default_params(b_transposed=1)
    with pytest.raises(fpsk.FpskError):
        fpsk.probe(dA, dB, dC, fpsk.probe_workspace(n, n, n), fpsk.new_probe_result(), None, p)
    with pytest.raises(fpsk.FpskError):
        fpsk.verify_repair(dA, dB, dC, 1, fpsk.repair_workspace(n, n, n, 0, fpsk.default_params()), 0, p)
