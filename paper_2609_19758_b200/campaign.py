"""Recovery campaign over the benchmark configurations (``python -m paper_2609_19758_b200.campaign``).

Runs, on seeded synthetic products (the vendor FP32-output GEMM delivers C), the whole verifier as a user
would: noise measurement on the clean product -> plan, both probes on the clean and on the faulty product,
localization at the planned bucket count and radius.  Counts, per fault population, how many injected
faults were reported, how many clean entries were reported (must be 0: Lemma 1), how often the probes
fired, and prints Wilson 95 % intervals.  One JSON line per case, then one summary line.

  config 1  256^3 FP16, U(-1,1): one clean product and three with one fault of 0.5 rms(C)
  config 2  4096^3 BF16, N(0,1) x N(0,1/sqrt k): four faults of 2-9 % rms(C); 20 seeds
  config 3  transformer layer shapes, FP16 and BF16: four faults of 1 rms(C) and four of 2-9 % each
  config 4  8192^3 FP16, U(-1,1): sixteen simultaneous faults, four sharing a row and three a column,
            half exponent-flip sized; 10 seeds
"""
from __future__ import annotations

import argparse
import json
import math

import torch

from . import build as B
from . import fpsk, harness, workloads as W


def _print_line(line: str) -> None:
    print(line, flush=True)


EMIT = _print_line          # where the per-case JSON lines go (a caller that owns stdout redirects them)


def wilson(k: int, n: int, z: float = 1.959964):
    if n == 0:
        return None
    p = k / n
    d = 1.0 + z * z / n
    c = (p + z * z / (2 * n)) / d
    h = z * math.sqrt(p * (1 - p) / n + z * z / (4 * n * n)) / d
    return [max(0.0, c - h), min(1.0, c + h)]


def line_population(faults):
    """'shared' for faults that share their row or column with another one of the same product."""
    rows, cols = {}, {}
    for f in faults:
        rows[f.i] = rows.get(f.i, 0) + 1
        cols[f.j] = cols.get(f.j, 0) + 1
    return [rows[f.i] > 1 or cols[f.j] > 1 for f in faults]


def run_case(tag, kind, n1, n2, n3, dtype, seed, make_faults, params, probe_buckets, tally):
    A, Bm = W.operands(kind, n1, n2, n3, dtype, seed)
    dA, dB = A.cuda(), Bm.cuda()
    dC = harness.vendor_gemm_fp32(dA, dB)
    rms = float(torch.sqrt(torch.mean(dC.double() ** 2)))
    ws0 = fpsk.workspace(n1, n2, n3, 0, params)
    nz = fpsk.measure_noise(dA, dB, dC, seed, ws0, 0, params)
    del ws0
    faults = make_faults(dC, rms)
    dCf = dC.clone()
    for f in faults:
        if f.kind == "add":
            dCf[f.i, f.j] += f.value
        else:
            dCf[f.i, f.j] *= 2.0 ** f.value
    pws = fpsk.probe_workspace(n1, n2, n3)
    res = fpsk.new_probe_result()
    fpsk.probe(dA, dB, dC, pws, res, None, params)
    r_c = fpsk.read_probe_result(res)
    clean_fired = r_c.fired
    dirty_fired = None
    if faults:
        fpsk.probe(dA, dB, dCf, pws, res, None, params)
        dirty_fired = fpsk.read_probe_result(res).fired
    hp = fpsk.HashedProbe(n1, n2, n3, probe_buckets, seed=seed + 1000)
    hp(dA, dB, dC, res, params=params)
    r_h = fpsk.read_probe_result(res)
    h_clean = r_h.fired
    h_dirty = None
    if faults:
        hp(dA, dB, dCf, res, params=params)
        h_dirty = fpsk.read_probe_result(res).fired
    p = fpsk.default_params()
    for name, _ in fpsk.Params._fields_:
        setattr(p, name, getattr(params, name))
    p.radius = nz.radius
    ws = fpsk.workspace(n1, n2, n3, nz.m_loc, p)
    got = fpsk.localize(dA, dB, dCf, seed, nz.m_loc, ws, p)
    got_clean = fpsk.localize(dA, dB, dC, seed, nz.m_loc, ws, p) if faults else got
    want = {(f.i, f.j) for f in faults}
    have = {(f.i, f.j) for f in got}
    shared = line_population(faults)
    for f, sh in zip(faults, shared):
        hit = (f.i, f.j) in have
        for pop in [f.population] + (["shared-line"] if sh else []):
            t = tally.setdefault(pop, [0, 0])
            t[0] += int(hit)
            t[1] += 1
    tally["false-positive entries"] = tally.get("false-positive entries", 0) + len(have - want) + len(got_clean)
    tally.setdefault("probe fired on clean", [0, 0])
    tally["probe fired on clean"][0] += int(clean_fired)
    tally["probe fired on clean"][1] += 1
    tally.setdefault("hashed probe fired on clean", [0, 0])
    tally["hashed probe fired on clean"][0] += int(h_clean)
    tally["hashed probe fired on clean"][1] += 1
    if faults:
        for key, v in (("probe fired on faulty", dirty_fired), ("hashed probe fired on faulty", h_dirty)):
            tally.setdefault(key, [0, 0])
            tally[key][0] += int(v)
            tally[key][1] += 1
    EMIT(json.dumps(dict(case=tag, shape=[n1, n2, n3], dtype="fp16" if dtype == W.FP16 else "bf16", seed=seed,
                          c_hat=nz.c_hat, plan=[nz.m0, nz.m_loc, nz.radius], injected=len(faults), found=len(want & have),
                          false_positives=len(have - want) + len(got_clean), probe=[int(clean_fired), dirty_fired],
                          hashed_probe=[int(h_clean), h_dirty],
                          probe_clean=dict(max_abs=r_c.max_abs, sigma_hat=r_c.sigma_hat, thr=r_c.thr, tau=r_c.tau),
                          hashed_clean=dict(m=probe_buckets, max_abs=r_h.max_abs, sigma_hat=r_h.sigma_hat, thr=r_h.thr,
                                            tau=r_h.tau))))
    del ws, dA, dB, dC, dCf
    torch.cuda.empty_cache()


def run(configs=(1, 2, 3, 4), seeds2=20, seeds4=10, tensor_cores=1, probe_buckets=256, shapes3=None):
    """Runs the chosen configurations and returns the summary (per-population recovery, false positives, probes)."""
    B.build()
    fpsk.lib()
    todo = set(configs)
    tally = {}
    tc = tensor_cores
    if 1 in todo:
        p = fpsk.default_params(s_budget=1, delta_max=1, tensor_cores=tc)
        run_case("cfg1", "uniform", 256, 256, 256, W.FP16, 1, lambda dC, rms: [], p, 16, tally)
        for s in (1, 2, 3):
            run_case("cfg1", "uniform", 256, 256, 256, W.FP16, 1,
                     lambda dC, rms, s=s: W.faults_additive(256, 256, rms, s, 1, 0.5, 0.5, "typical"), p, 16, tally)
    if 2 in todo:
        p = fpsk.default_params(s_budget=4, tensor_cores=tc)
        for s in range(seeds2):
            run_case("cfg2", "gauss_scaled", 4096, 4096, 4096, W.BF16, s,
                     lambda dC, rms, s=s: W.faults_additive(4096, 4096, rms, s, 4, 0.02, 0.09, "small"), p,
                     probe_buckets, tally)
    if 3 in todo:
        p = fpsk.default_params(tensor_cores=tc)
        for (n1, n2, n3) in (shapes3 if shapes3 is not None else W.TRANSFORMER_SHAPES):
            for dt in (W.FP16, W.BF16):
                def mk(dC, rms, n1=n1, n3=n3):
                    a = W.faults_additive(n1, n3, rms, 7, 4, 1.0, 1.0, "typical")
                    b = W.faults_additive(n1, n3, rms, 8, 4, 0.02, 0.09, "small", taken=[(f.i, f.j) for f in a])
                    return a + b
                run_case("cfg3", "transformer", n1, n2, n3, dt, 7, mk, p, probe_buckets, tally)
    if 4 in todo:
        p = fpsk.default_params(s_budget=16, delta_max=4, tensor_cores=tc)
        for s in range(seeds4):
            run_case("cfg4", "uniform", 8192, 8192, 8192, W.FP16, s,
                     lambda dC, rms, s=s: W.faults_mixed16(dC.cpu(), rms, s), p, probe_buckets, tally)
    summary = {}
    for k, v in tally.items():
        if isinstance(v, list):
            summary[k] = dict(hits=v[0], of=v[1], rate=(v[0] / v[1]) if v[1] else None, wilson95=wilson(v[0], v[1]))
        else:
            summary[k] = v
    return summary


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--configs", default="1,2,3,4")
    ap.add_argument("--seeds2", type=int, default=20)
    ap.add_argument("--seeds4", type=int, default=10)
    ap.add_argument("--tensor-cores", type=int, default=1, choices=[0, 1])
    ap.add_argument("--probe-buckets", type=int, default=256)
    args = ap.parse_args()
    torch.cuda.set_device(0)
    summary = run({int(x) for x in args.configs.split(",")}, args.seeds2, args.seeds4, args.tensor_cores, args.probe_buckets)
    print(json.dumps(dict(summary=summary, tensor_cores=args.tensor_cores, probe_buckets=args.probe_buckets)))


if __name__ == "__main__":
    main()
