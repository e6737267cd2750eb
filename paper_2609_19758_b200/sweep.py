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
    for i in range(iters):
        flush.max()                     # evict L2 with a read; also keeps the GPU busy before the timed call
        evs[i][0].record()
        fn()
        evs[i][1].record()
    torch.cuda.synchronize()
    ts = sorted(a.elapsed_time(b) for a, b in evs)
    return ts[len(ts) // 2], ts[0]


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--sizes", default="1024,2048,4096,8192,16384")
    ap.add_argument("--iters", type=int, default=20)
    ap.add_argument("--tensor-cores", type=int, default=0, choices=[0, 1],
                    help="contraction of the moment sketches: 1 = split-BF16 tcgen05 at >= 384 buckets")
    args = ap.parse_args()
    B.build()
    fpsk.lib()
    torch.cuda.set_device(0)
    flush = torch.zeros(64 << 20, dtype=torch.int32, device="cuda")
    gen = torch.Generator(device="cuda")
    rows = []
    for dt_name, dt in (("bf16", torch.bfloat16), ("fp16", torch.float16)):
        for n in [int(x) for x in args.sizes.split(",")]:
            gen.manual_seed(1000 + n)
            A = torch.randn(n, n, device="cuda", generator=gen).to(dt)
            Bm = torch.randn(n, n, device="cuda", generator=gen).to(dt)
            C = harness.vendor_gemm_fp32(A, Bm)
            d = fpsk.BF16 if dt == torch.bfloat16 else fpsk.FP16
            p = fpsk.default_params(tensor_cores=args.tensor_cores)
            ws0 = fpsk.workspace(n, n, n, 0, p)
            nz = fpsk.measure_noise(A, Bm, C, 7, ws0, 0, p)
            pws = fpsk.probe_workspace(n, n, n)
            res = fpsk.new_probe_result()
            it = args.iters if n <= 8192 else max(5, args.iters // 2)
            probe_ms, probe_min = _time(lambda: fpsk.probe(A, Bm, C, pws, res, None, p), it, flush)
            verdict = fpsk.read_probe_result(res)
            gemm_ms, _ = _time(lambda: harness.vendor_gemm_fp32(A, Bm), it, flush)
            noise_ms, _ = _time(lambda: fpsk.measure_noise(A, Bm, C, 7, ws0, 0, p), max(3, it // 4), flush)
            del ws0
            p.radius = nz.radius
            m_loc = min(nz.m_loc, fpsk.max_buckets(n, n, n))
            ws = fpsk.workspace(n, n, n, m_loc, p)
            found = []
            loc_ms, _ = _time(lambda: found.append(len(fpsk.localize(A, Bm, C, 7, m_loc, ws, p))), max(3, it // 4), flush)
            nbytes = 2 * n * n + 2 * n * n + 4 * n * n
            row = dict(n=n, dtype=dt_name, tensor_cores=args.tensor_cores, c_hat=nz.c_hat, sigma_clip=nz.sigma_clip, sigma_mad=nz.sigma_mad, rms_c=nz.rms_c,
                       m0=nz.m0, m_probe=nz.m_probe, m_loc=nz.m_loc, radius=nz.radius, probe_ms=probe_ms, probe_ms_min=probe_min,
                       probe_gbs=nbytes / probe_ms / 1e6, gemm_ms=gemm_ms, measure_noise_ms=noise_ms, localize_ms=loc_ms,
                       clean_fired=int(verdict.fired), clean_faults_reported=max(found) if found else 0)
            rows.append(row)
            print(json.dumps(row), flush=True)
            del ws, A, Bm, C
            torch.cuda.empty_cache()
    fits = {}
    for dt_name in ("bf16", "fp16"):
        pts = [(math.log(r["n"]), math.log(r["c_hat"])) for r in rows if r["dtype"] == dt_name and r["c_hat"] > 0]
        if len(pts) >= 2:
            mx = statistics.mean(x for x, _ in pts)
            my = statistics.mean(y for _, y in pts)
            e = sum((x - mx) * (y - my) for x, y in pts) / sum((x - mx) ** 2 for x, _ in pts)
            fits[dt_name] = dict(exponent_of_n_beyond_1p5=e, c_hat_at_4096=math.exp(my + e * (math.log(4096) - mx)))
    print(json.dumps(dict(fit=fits)))


if __name__ == "__main__":
    main()
