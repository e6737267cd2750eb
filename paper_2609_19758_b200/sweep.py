"""Clean-path noise and cost sweep on square products (``python -m paper_2609_19758_b200.sweep``).

For n in {1024, 2048, 4096, 8192, 16384} and both operand types (A, B ~ N(0,1), FP32 C from the
vendor GEMM, no faults): measures the sketch-noise constant c_hat at the law's bucket count,
fits its exponent in n, derives the plan (m_loc, r), and times the probe, the noise
measurement, a localization forced on the clean product and the vendor GEMM.  Operands are
drawn on the device (torch generator, seeded) because the largest case is 2 GB of inputs.
Prints one JSON line per case and a final line with the fits.
"""
from __future__ import annotations

import argparse
import json
import math
import statistics

import torch

from . import build as B
from . import fpsk, harness


def _time(fn, iters, flush):
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(iters)]
    for _ in range(2):                  # untimed: first-call set-up (kernel attributes, pooled streams, first touch of the workspace)
        fn()
    for i in range(iters):
        flush.max()                     # evict L2 with a read; also keeps the GPU busy before the timed call
        evs[i][0].record()
        fn()
        evs[i][1].record()
    torch.cuda.synchronize()
    ts = sorted(a.elapsed_time(b) for a, b in evs)
    return ts[len(ts) // 2], ts[0]


def _burst(fn_for, nsets, launches=30, reps=3):
    """Average duration of one call when `launches` of them run back to back from a CUDA graph over rotating
    input batches (each larger than L2, so every launch still reads its operands from HBM): the launch duration
    without the cost of an event pair per launch."""
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        for i in range(launches):
            fn_for(i % nsets)()
    best = None
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for _ in range(reps + 1):
        torch.cuda.synchronize()
        e0.record()
        g.replay()
        e1.record()
        torch.cuda.synchronize()
        t = e0.elapsed_time(e1) / launches
        best = t if best is None else min(best, t)
    return best


def run(sizes=(1024, 2048, 4096, 8192, 16384), iters=20, tensor_cores=0, dtypes=("bf16", "fp16"), emit=None,
        with_localize=True):
    """Rows of the sweep (one dict per size and operand type) and the fitted exponents."""
    B.build()
    fpsk.lib()
    flush = torch.zeros(64 << 20, dtype=torch.int32, device="cuda")
    gen = torch.Generator(device="cuda")
    rows = []
    for dt_name in dtypes:
        dt = torch.bfloat16 if dt_name == "bf16" else torch.float16
        for n in sizes:
            nbytes = 2 * n * n + 2 * n * n + 4 * n * n
            # batches for the back-to-back figure: each must exceed L2 (126 MB), three of them rotate
            nsets = 3 if nbytes >= 128e6 and n <= 8192 else (2 if nbytes >= 128e6 else 1)
            sets = []
            for q in range(nsets):
                gen.manual_seed(1000 + n + 7919 * q)
                A = torch.randn(n, n, device="cuda", generator=gen).to(dt)
                Bm = torch.randn(n, n, device="cuda", generator=gen).to(dt)
                sets.append((A, Bm, harness.vendor_gemm_fp32(A, Bm)))
            A, Bm, C = sets[0]
            p = fpsk.default_params(tensor_cores=tensor_cores)
            # one workspace for the measurement and the localization, sized for the largest bucket count the plan can ask
            # for (as bench.py does): the measurement then has room to transpose B once instead of compressing it as k x n
            mb_cap = min(fpsk.max_buckets(n, n, n), max(16, int((n * n // 16) ** 0.5)))
            mb_cap = max(mb_cap, fpsk.law_m_start(n, n, n, dt_name == "bf16" and 1 or 0, p))
            ws0 = fpsk.workspace(n, n, n, mb_cap, p)
            nz = fpsk.measure_noise(A, Bm, C, 7, ws0, 0, p)
            pws = fpsk.probe_workspace(n, n, n)
            res = fpsk.new_probe_result()
            it = iters if n <= 8192 else max(5, iters // 2)
            probe_ms, probe_min = _time(lambda: fpsk.probe(A, Bm, C, pws, res, None, p), it, flush)
            verdict = fpsk.read_probe_result(res)
            burst_ms = None
            if nsets >= 2:
                burst_ms = _burst(lambda q: (lambda: fpsk.probe(sets[q][0], sets[q][1], sets[q][2], pws, res, None, p)), nsets)
            gemm_ms, _ = _time(lambda: harness.vendor_gemm_fp32(A, Bm), it, flush)
            noise_ms, _ = _time(lambda: fpsk.measure_noise(A, Bm, C, 7, ws0, 0, p), max(3, it // 4), flush)
            row = dict(n=n, dtype=dt_name, tensor_cores=tensor_cores, c_hat=nz.c_hat, sigma_clip=nz.sigma_clip, sigma_mad=nz.sigma_mad,
                       rms_c=nz.rms_c, m0=nz.m0, m_probe=nz.m_probe, m_loc=nz.m_loc, radius=nz.radius, probe_ms=probe_ms,
                       probe_ms_min=probe_min, probe_gbs=nbytes / probe_ms / 1e6, probe_ms_burst=burst_ms,
                       probe_gbs_burst=(nbytes / burst_ms / 1e6) if burst_ms else None, gemm_ms=gemm_ms,
                       measure_noise_ms=noise_ms, clean_fired=int(verdict.fired))
            if with_localize:
                p.radius = nz.radius
                m_loc = min(nz.m_loc, mb_cap)
                found = []
                loc_ms, _ = _time(lambda: found.append(len(fpsk.localize(A, Bm, C, 7, m_loc, ws0, p))), max(3, it // 4), flush)
                row.update(localize_ms=loc_ms, clean_faults_reported=max(found) if found else 0)
            del ws0
            rows.append(row)
            if emit:
                emit(row)
            del sets, A, Bm, C
            torch.cuda.empty_cache()
    fits = {}
    for dt_name in dtypes:
        pts = [(math.log(r["n"]), math.log(r["c_hat"])) for r in rows if r["dtype"] == dt_name and r["c_hat"] > 0]
        if len(pts) >= 2:
            mx = statistics.mean(x for x, _ in pts)
            my = statistics.mean(y for _, y in pts)
            e = sum((x - mx) * (y - my) for x, y in pts) / sum((x - mx) ** 2 for x, _ in pts)
            fits[dt_name] = dict(exponent_of_n_beyond_1p5=e, c_hat_at_4096=math.exp(my + e * (math.log(4096) - mx)))
    return rows, fits


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--sizes", default="1024,2048,4096,8192,16384")
    ap.add_argument("--iters", type=int, default=20)
    ap.add_argument("--tensor-cores", type=int, default=0, choices=[0, 1],
                    help="contraction of the moment sketches: 1 = split-FP16 tcgen05 at >= 384 buckets")
    args = ap.parse_args()
    torch.cuda.set_device(0)
    rows, fits = run([int(x) for x in args.sizes.split(",")], args.iters, args.tensor_cores,
                     emit=lambda r: print(json.dumps(r), flush=True))
    print(json.dumps(dict(fit=fits)))


if __name__ == "__main__":
    main()
