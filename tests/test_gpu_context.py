"""Caller-owned host resources: with a context in fpsk_params the noise measurement, the localization and the
whole verify-and-repair path create nothing themselves (no stream, event or pinned buffer) and return exactly
what they return with the library's own lazily created set."""
import numpy as np
import pytest
import torch

from paper_2609_19758_b200 import build as B
from paper_2609_19758_b200 import fpsk, harness, workloads as W

pytestmark = pytest.mark.gpu


def _faults(got):
    return [(f.i, f.j, f.delta, f.recompute, f.c_value, f.round, f.bucket_a, f.bucket_b) for f in got]


@pytest.mark.parametrize("tensor_cores", [0, 1])
def test_context_gives_the_same_results_and_creates_nothing(tensor_cores):
    B.build()
    n = 1024
    A, Bm = W.operands("gauss_scaled", n, n, n, W.BF16, 5)
    dA, dB = A.cuda(), Bm.cuda()
    dC = harness.vendor_gemm_fp32(dA, dB)
    rms = float(torch.sqrt(torch.mean(dC.double() ** 2)))
    faults = W.faults_additive(n, n, rms, 5, 4, 0.05, 0.5, "small")
    dCf = dC.clone()
    for f in faults:
        dCf[f.i, f.j] += f.value
    m_b = 384 if tensor_cores else 64
    out = []
    with fpsk.Context() as ctx:
        for use_ctx in (False, True):
            p = fpsk.default_params(s_budget=4, tensor_cores=tensor_cores, radius=3)
            p.context = ctx.ptr if use_ctx else None
            before = fpsk.lazy_resource_count()
            ws = fpsk.workspace(n, n, n, m_b, p)
            nz = fpsk.measure_noise(dA, dB, dC, 9, ws, m_b, p)
            got = fpsk.localize(dA, dB, dCf, 9, m_b, ws, p)
            rws = fpsk.repair_workspace(n, n, n, m_b, p)
            Cr = dCf.clone()
            rep_f, rep = fpsk.verify_repair(dA, dB, Cr, 9, rws, m_b, p)
            torch.cuda.synchronize()
            if use_ctx:
                assert fpsk.lazy_resource_count() == before          # nothing created behind the caller's back
            out.append(((nz.sigma_clip, nz.sigma_mad, nz.rms_c, nz.m_loc, nz.radius), _faults(got), _faults(rep_f),
                        (rep.state, rep.n_faults), Cr.clone()))
            del ws, rws
    assert out[0][0] == out[1][0] and out[0][1] == out[1][1] and out[0][2] == out[1][2] and out[0][3] == out[1][3]
    assert torch.equal(out[0][4], out[1][4])
    assert {(f[0], f[1]) for f in out[1][1]} == {(f.i, f.j) for f in faults}
    assert out[1][3][0] == 1


def test_context_of_another_device_is_refused_and_destroy_accepts_null():
    B.build()
    assert fpsk.lib().fpsk_context_destroy(None) == 0
    assert fpsk.lib().fpsk_context_create(None) == fpsk.ERR_NULL
