"""fpsk_probe_static: the probe for callers that cannot allocate device memory.

Such callers (code inside a stream capture, a latency-critical or fault-handling path that
must stay out of the allocator, a plug-in that owns no memory pool) get the probe's scratch
from a fixed array inside the library.  The test calls the entry point through the C ABI twice
in a row and checks each result against fpsk_probe with a caller-owned workspace: the kernel
is the same and its summation order is fixed, so the two must agree bit for bit, which is well
inside the 1e-5 tolerance the other probe tests use.  The second call runs on a different
product, so it also shows that nothing stale from the first call leaks into it.  The residual
is also held against the definition (column sums of E = AB - C in FP64) like in the other
probe tests.
"""
import ctypes as C

import numpy as np
import oracle as O
import pytest
import torch

from paper_2609_19758_b200 import build as B
from paper_2609_19758_b200 import fpsk, harness, workloads as W

pytestmark = pytest.mark.gpu


def _fields(r):
    return (r.fired, r.nonfinite, r.argmax_col, r.status, r.max_abs, r.sigma_hat, r.thr, r.tau)


def test_probe_static_matches_probe_on_two_calls_in_a_row():
    B.build()
    n1, n2, n3 = 512, 768, 1024
    cases, hosts = [], []
    for seed in (3, 4):
        A, Bm = W.operands("gauss_scaled", n1, n2, n3, W.BF16, seed)
        dA, dB = A.cuda(), Bm.cuda()
        dC = harness.vendor_gemm_fp32(dA, dB)
        cases.append((dA, dB, dC))
        hosts.append((A, Bm))
    # the second product carries a fault, so the two calls must give different verdicts
    cases[1][2][17, 33] += 0.25

    ws = fpsk.probe_workspace(n1, n2, n3)
    want = []
    for dA, dB, dC in cases:
        res = fpsk.new_probe_result()
        resid = torch.empty(n3, dtype=torch.float32, device="cuda")
        fpsk.probe(dA, dB, dC, ws, res, resid)
        torch.cuda.synchronize()
        want.append((fpsk.read_probe_result(res), resid.clone()))

    got = []
    for dA, dB, dC in cases:          # two calls in a row on the shared built-in scratch
        res = fpsk.new_probe_result()
        resid = torch.empty(n3, dtype=torch.float32, device="cuda")
        fpsk.probe_static(dA, dB, dC, res, resid)
        got.append((res, resid))
    torch.cuda.synchronize()

    for (w_res, w_resid), (g_res, g_resid) in zip(want, got):
        g = fpsk.read_probe_result(g_res)
        assert g.status == 0
        scale = float(w_resid.abs().max()) + 1.0
        assert float((g_resid - w_resid).abs().max()) <= 1e-5 * scale
        assert torch.equal(g_resid, w_resid)              # same kernel, fixed order: identical
        assert _fields(g) == _fields(w_res)
    for (A, Bm), (_, _, dC), (g_res, g_resid) in zip(hosts, cases, got):
        A64, B64 = A.double().numpy(), Bm.double().numpy()
        E = O.error_matrix(A64, B64, dC.cpu().numpy())
        abs_j = O.abs_product(A64, B64).sum(axis=0)
        assert np.all(np.abs(g_resid.cpu().double().numpy() - O.probe_sketch(E)) <= 1e-5 * abs_j)
        g = fpsk.read_probe_result(g_res)
        v = O.probe_verdict(O.probe_sketch(E), O.analytic_tau(A64, B64, n2), n_rows=n1)
        assert bool(g.fired) == v.fired
    assert fpsk.read_probe_result(got[0][0]).fired == 0
    assert fpsk.read_probe_result(got[1][0]).fired == 1 and fpsk.read_probe_result(got[1][0]).argmax_col == 33


def test_probe_static_refuses_what_does_not_fit_or_is_not_fp32():
    B.build()
    L = fpsk.lib()
    one = C.c_void_p(4096)        # never dereferenced: the checks come first
    # a shape whose scratch exceeds the built-in array
    big = 1 << 22
    assert L.fpsk_probe_workspace_bytes(big, big, big) > fpsk.PROBE_STATIC_SCRATCH_BYTES
    assert L.fpsk_probe_static(one, big, one, big, one, big, big, big, big, 1, 1, None, None, one, None) == fpsk.ERR_WORKSPACE
    # a narrowed C is rejected like in fpsk_probe
    assert L.fpsk_probe_static(one, 8, one, 8, one, 8, 8, 8, 8, 1, 0, None, None, one, None) == fpsk.ERR_DTYPE
    assert L.fpsk_probe_static(None, 8, one, 8, one, 8, 8, 8, 8, 1, 1, None, None, one, None) == fpsk.ERR_NULL
