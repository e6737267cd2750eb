"""Run to run, bit for bit: the verifier has no float atomics and fixed orders of addition, and its side streams
are joined by events, so repeated calls on the same inputs (and on a workspace left dirty by other calls) must
return identical numbers.  A race between its streams would show up here as an occasional different value."""
import pytest
import torch

from paper_2609_19758_b200 import build as B
from paper_2609_19758_b200 import fpsk, harness, workloads as W

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _lib():
    B.build()
    fpsk.lib()


def _noise_fields(nz):
    return tuple(getattr(nz, name) for name, _ in fpsk.Noise._fields_)


@pytest.mark.parametrize("tc,m_b", [(0, 0), (1, 512)])
def test_noise_measurement_and_localization_repeat_exactly(tc, m_b):
    n1, n2, n3 = 1536, 1024, 2048
    A, Bm = W.operands("gauss_scaled", n1, n2, n3, W.BF16, 19)
    dA, dB = A.cuda(), Bm.cuda()
    dC = harness.vendor_gemm_fp32(dA, dB)
    faults = W.faults_additive(n1, n3, W.rms(dC.cpu()), 2, 4, 0.05, 0.5, "typical")
    dF = W.inject(dC.cpu(), faults)[0].cuda()
    p = fpsk.default_params(s_budget=4, radius=4, tensor_cores=tc)
    m_loc = m_b if m_b else 384
    ws = fpsk.workspace(n1, n2, n3, m_loc, p)
    first_noise = first_loc = None
    for it in range(40):
        if it % 7 == 3:
            ws.random_(0, 255)                      # whatever another call may have left behind
        nz = _noise_fields(fpsk.measure_noise(dA, dB, dC, 5, ws, m_b, p))
        got = [(f.i, f.j, f.delta, f.round, f.bucket_a, f.bucket_b) for f in fpsk.localize(dA, dB, dF, 9, m_loc, ws, p)]
        if first_noise is None:
            first_noise, first_loc = nz, got
            assert {(i, j) for (i, j, *_r) in got} == {(f.i, f.j) for f in faults}
        assert nz == first_noise, it
        assert got == first_loc, it


def test_two_host_threads_share_the_pools():
    """Concurrent calls from two threads on their own streams and workspaces: each leases its own auxiliary streams
    and staging buffer."""
    import threading
    n = 1024
    A, Bm = W.operands("gauss_scaled", n, n, n, W.FP16, 23)
    dA, dB = A.cuda(), Bm.cuda()
    dC = harness.vendor_gemm_fp32(dA, dB)
    p = fpsk.default_params(tensor_cores=1, radius=3)
    ref_ws = fpsk.workspace(n, n, n, 384, p)
    ref = _noise_fields(fpsk.measure_noise(dA, dB, dC, 5, ref_ws, 384, p))
    ref_loc = fpsk.localize(dA, dB, dC, 5, 384, ref_ws, p)
    assert ref_loc == []
    errors = []

    def work(k):
        try:
            st = torch.cuda.Stream()
            ws = fpsk.workspace(n, n, n, 384, p)
            for _ in range(15):
                nz = _noise_fields(fpsk.measure_noise(dA, dB, dC, 5, ws, 384, p, stream=st))
                if nz != ref:
                    errors.append((k, nz))
                if fpsk.localize(dA, dB, dC, 5, 384, ws, p, stream=st) != []:
                    errors.append((k, "faults on a clean product"))
        except Exception as e:      # noqa: BLE001 - reported through the list
            errors.append((k, repr(e)))

    ts = [threading.Thread(target=work, args=(k,)) for k in range(2)]
    for t in ts:
        t.start()
    for t in ts:
        t.join()
    assert not errors, errors[:3]
