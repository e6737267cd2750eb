"""The index-checked build of the library (libfpsk_bounds.so, -DFPSK_DEBUG_BOUNDS) runs the odd-shaped small cases -
unaligned leading dimensions, sizes that are no multiple of any tile, ragged last buckets - through every entry point
and must record no index out of range.  (Every index a kernel takes from a table is checked there before it addresses
memory; a violation is recorded and the access skipped, so the process carries on and reports it.)  The cases run in
a child process because a process loads one build of the library."""
import json
import os
import subprocess
import sys

import pytest

from paper_2609_19758_b200 import build as B

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r"""
import json, sys
import numpy as np, torch
from paper_2609_19758_b200 import fpsk, harness, workloads as W
rep0 = fpsk.debug_bounds_report()
done = []
for (n1, n2, n3, dt, m_b) in [(77, 33, 255, W.FP16, 16), (300, 40, 520, W.BF16, 64), (1000, 72, 1536, W.FP16, 384),
                               (513, 264, 1030, W.BF16, 96)]:
    A, Bm = W.operands("integer", n1, n2, n3, dt, 3, lim=6)
    Cm = W.cpu_fp32_product(A, Bm)
    coords = [(n1 - 1, n3 - 1), (0, 0), (n1 // 2, n3 // 3)]
    Cf = Cm.clone()
    for t, (i, j) in enumerate(coords):
        Cf[i, j] += float(3 + t)
    # views with leading dimensions that are no multiple of 8: the unaligned code paths
    pad = lambda X, extra: torch.nn.functional.pad(X, (0, extra))[:, :X.shape[1]]
    dA, dB, dC = pad(A.cuda(), 3), pad(Bm.cuda(), 5), pad(Cf.cuda(), 1)
    for tc in (0, 1):
        p = fpsk.default_params(radius=2, tensor_cores=tc, s_budget=4)
        pws = fpsk.probe_workspace(n1, n2, n3); res = fpsk.new_probe_result()
        fpsk.probe(dA, dB, dC, pws, res, None, p)
        fired = fpsk.read_probe_result(res).fired
        ws = fpsk.workspace(n1, n2, n3, m_b, p)
        fpsk.sketches(dA, dB, dC, 5, 0, m_b, ws, params=p)
        nz = fpsk.measure_noise(dA, dB, dC, 5, ws, m_b, p)
        got = fpsk.localize(dA, dB, dC, 5, m_b, ws, p)
        Wt = Bm.t().contiguous().cuda()
        pt = fpsk.default_params(radius=2, tensor_cores=tc, s_budget=4, b_transposed=1)
        got_t = fpsk.localize(dA, Wt, dC, 5, m_b, fpsk.workspace(n1, n2, n3, m_b, pt), pt)
        rws = fpsk.repair_workspace(n1, n2, n3, m_b, p)
        Cr = Cf.cuda().clone()
        _, rrep = fpsk.verify_repair(A.cuda(), Bm.cuda(), Cr, 5, rws, m_b, p)
        hp = fpsk.HashedProbe(n1, n2, n3, min(m_b, 64), seed=9)
        hp(dA, dB, dC, res)
        # contiguous operands: where the sizes allow, the bulk-copy kernels (with tc = 1 the single-launch form)
        hp2 = fpsk.HashedProbe(n1, n2, n3, min(m_b, 64), seed=9)
        hp2(A.cuda(), Bm.cuda(), Cf.cuda(), res, params=p)
        torch.cuda.synchronize()
        fired = fired and fpsk.read_probe_result(res).fired and fpsk.read_probe_result(res).status == 0
        done.append(dict(shape=[n1, n2, n3], tc=tc, fired=int(fired), found=sorted((f.i, f.j) for f in got) == sorted(coords),
                         found_t=sorted((f.i, f.j) for f in got_t) == sorted(coords), repaired=int(rrep.state == 1),
                         restored=bool(torch.equal(Cr.cpu(), Cm))))
print(json.dumps(dict(before=rep0, after=fpsk.debug_bounds_report(), cases=done)))
"""


def test_odd_shapes_record_no_index_out_of_range():
    lib = B.build(bounds=True)
    env = dict(os.environ, FPSK_LIBRARY=lib, PYTHONPATH=ROOT + os.pathsep + os.environ.get("PYTHONPATH", ""))
    out = subprocess.run([sys.executable, "-c", CHILD], env=env, cwd=ROOT, capture_output=True, text=True, timeout=900)
    assert out.returncode == 0, out.stderr[-3000:]
    rep = json.loads(out.stdout.strip().splitlines()[-1])
    assert rep["before"][0] == 1 and rep["before"][1] == 0          # the checked build is the one that ran
    built, violations, line, index, limit, src = rep["after"]
    assert built == 1 and violations == 0, (violations, src, line, index, limit)
    assert len(rep["cases"]) == 8
    for c in rep["cases"]:
        assert c["fired"] == 1 and c["found"] and c["found_t"] and c["repaired"] == 1 and c["restored"], c


def test_product_build_reports_that_it_has_no_checks():
    from paper_2609_19758_b200 import fpsk
    B.build()
    built, violations = fpsk.debug_bounds_report()[:2]
    if os.environ.get("FPSK_LIBRARY"):
        pytest.skip("another build of the library is loaded")
    assert built == 0 and violations == -1
