"""Host-side checks of the C ABI that need no GPU: the library loads, exports every symbol the
header declares, validates arguments before touching CUDA, and its scalar planner agrees with
the oracle's, which is pinned to the paper's printed values."""
import ctypes as C
import math
import os
import re

import pytest

import oracle as O
from paper_2609_19758_b200 import build as B
from paper_2609_19758_b200 import fpsk

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    B.build()
    return fpsk.lib()


def test_exports_every_declared_symbol(lib):
    names = set()
    for h in sorted(os.listdir(os.path.join(ROOT, "include"))):
        if not h.endswith(".h"):
            continue
        hdr = open(os.path.join(ROOT, "include", h)).read()
        hdr = re.sub(r"/\*.*?\*/", "", hdr, flags=re.S)
        names |= set(re.findall(r"\b(fpsk_[a-z_0-9]+)\s*\(", hdr))
    assert {"fpsk_probe", "fpsk_localize", "fpsk_measure_noise", "fpsk_sketches", "fpsk_plan", "fpsk_context_create",
            "fpsk_context_destroy", "fpsk_selftest_bounded_wait", "fpsk_launch_count"} <= names
    for n in names:
        assert hasattr(lib, n), n


def test_struct_layouts_match_header():
    assert C.sizeof(fpsk.ProbeResult) == 32
    assert C.sizeof(fpsk.Fault) == 40 and fpsk.Fault.delta.offset == 8 and fpsk.Fault.bucket_b.offset == 36
    assert C.sizeof(fpsk.Params) == 88 and fpsk.Params.rho_min.offset == 40 and fpsk.Params.b_transposed.offset == 32
    assert fpsk.Params.context.offset == 80
    assert C.sizeof(fpsk.Noise) == 56


def test_defaults_and_status_strings(lib):
    p = fpsk.default_params()
    assert (p.rounds, p.r_star, p.r_max, p.radius, p.s_budget, p.delta_max, p.mad_of_abs) == (3, 4, 16, -1, 8, 8, 1)
    assert (p.rho_min, p.c_valid, p.mu, p.b_star, p.c_coll) == (0.02, 100.0, 4.0, 0.3, 2.0)
    assert fpsk.status_string(0) == "ok" and "FP32" in fpsk.status_string(fpsk.ERR_DTYPE)


def test_law_start_matches_printed_table(lib):
    gold = os.path.join(ROOT, "tests", "golden", "tab_rect_law_m.txt")
    for line in open(gold):
        line = line.split("#")[0].split()
        if not line:
            continue
        n1, n2, n3, mb, mf = map(int, line)
        assert fpsk.law_m_start(n1, n2, n3, fpsk.BF16) == mb
        assert fpsk.law_m_start(n1, n2, n3, fpsk.FP16) == mf
    assert fpsk.law_m_start(16384, 16384, 16384, fpsk.FP16) == 2397
    assert fpsk.law_m_start(256, 256, 256, fpsk.FP16, fpsk.default_params(s_budget=1, delta_max=1)) == 16
    assert fpsk.law_m_start(0, 4, 4, fpsk.FP16) == -1


def test_plan_matches_oracle_on_a_grid(lib):
    shapes = [(256, 256, 256), (4096, 4096, 4096), (2048, 11008, 4096), (4096, 4096, 11008), (8192, 8192, 8192),
              (16384, 16384, 16384), (7, 33, 255)]
    for (n1, n2, n3) in shapes:
        for dt in (fpsk.FP16, fpsk.BF16):
            for m_cur in (16, 48, 230, 1000):
                for sig in (1e-7, 3e-6, 1e-4, 2e-3, float("nan"), 0.0):
                    for rms in (1.0, 0.37, 12.0):
                        want = O.plan(n1, n2, n3, dt, sig, rms, m_cur)
                        got = fpsk.plan(n1, n2, n3, dt, sig, rms, m_cur)
                        assert got[:2] == want[:2], (n1, n2, n3, dt, m_cur, sig, rms)
                        assert got[2] == pytest.approx(want[2], rel=1e-12)


def test_argument_validation_needs_no_device(lib):
    p = fpsk.default_params()
    one = C.c_void_p(4096)          # never dereferenced: validation fails first
    f = lib.fpsk_probe
    assert f(one, 8, one, 8, one, 8, 8, 8, 8, 0, 0, None, one, 1 << 20, None, one, None) == fpsk.ERR_DTYPE  # C not FP32
    assert f(None, 8, one, 8, one, 8, 8, 8, 8, 0, 1, None, one, 1 << 20, None, one, None) == fpsk.ERR_NULL
    assert f(one, 8, one, 8, one, 8, 8, 8, 8, 7, 1, None, one, 1 << 20, None, one, None) == fpsk.ERR_DTYPE
    assert f(one, 4, one, 8, one, 8, 8, 8, 8, 0, 1, None, one, 1 << 20, None, one, None) == fpsk.ERR_SHAPE  # lda < k
    assert f(one, 8, one, 8, one, 8, 0, 8, 8, 0, 1, None, one, 1 << 20, None, one, None) == fpsk.ERR_SHAPE
    assert f(one, 8, one, 8, one, 8, 8, 8, 8, 0, 1, None, C.c_void_p(4097), 1 << 20, None, one, None) == fpsk.ERR_ALIGN
    bad = fpsk.default_params(rounds=0)
    assert f(one, 8, one, 8, one, 8, 8, 8, 8, 0, 1, C.byref(bad), one, 1 << 20, None, one, None) == fpsk.ERR_PARAM
    g = lib.fpsk_localize
    cnt = C.c_int32()
    buf = (fpsk.Fault * 4)()
    assert g(one, 8, one, 8, one, 8, 8, 8, 8, 0, 1, 0, None, one, 1 << 20, None, buf, 4, C.byref(cnt)) == fpsk.ERR_BUCKETS
    assert g(one, 8, one, 8, one, 8, 8, 8, 8, 0, 1, 4, None, one, 16, None, buf, 4, C.byref(cnt)) == fpsk.ERR_WORKSPACE
    # transposed weight (W = B^T, n x k): ldb is checked against k; only noise measurement and localization take it
    wt = fpsk.default_params(b_transposed=1)
    assert g(one, 8, one, 8, one, 16, 8, 8, 16, 0, 1, 4, C.byref(wt), one, 16, None, buf, 4, C.byref(cnt)) == fpsk.ERR_WORKSPACE
    assert g(one, 8, one, 8, one, 16, 8, 8, 16, 0, 1, 4, None, one, 16, None, buf, 4, C.byref(cnt)) == fpsk.ERR_SHAPE
    assert g(one, 16, one, 8, one, 8, 8, 16, 8, 0, 1, 4, C.byref(wt), one, 16, None, buf, 4, C.byref(cnt)) == fpsk.ERR_SHAPE
    assert f(one, 8, one, 8, one, 8, 8, 8, 8, 0, 1, C.byref(wt), one, 1 << 20, None, one, None) == fpsk.ERR_PARAM
    assert g(one, 8, one, 8, one, 8, 8, 8, 8, 0, 1, 4, C.byref(fpsk.default_params(b_transposed=2)), one, 1 << 20, None,
             buf, 4, C.byref(cnt)) == fpsk.ERR_PARAM
    assert lib.fpsk_hash_tables(1, 0, 2, 10, 4, one, one, None) == fpsk.ERR_PARAM
    assert lib.fpsk_probe_workspace_bytes(0, 1, 1) == 0
    assert lib.fpsk_probe_workspace_bytes(4096, 4096, 4096) > 0
    assert lib.fpsk_workspace_bytes(4096, 4096, 4096, 384, None) > 3 * 384 * 384 * 4
    assert lib.fpsk_workspace_bytes(4096, 4096, 4096, 10 ** 6, None) == 0
    assert fpsk.max_buckets(4096, 4096, 4096) >= 4096 and fpsk.max_buckets(16384, 16384, 16384) >= 4096


def test_bside_record_and_key_logic(lib):
    """The cache key of the B side (tensor identity and version; Section "Implementation") is host logic."""
    assert C.sizeof(fpsk.BSide) == 96 and fpsk.BSide.valid.offset == 76 and fpsk.BSide.built_transposed.offset == 88
    s = fpsk.BSide()
    Bp, cache = C.c_void_p(0x1000), C.c_void_p(0x2000)
    args = (Bp, 64, 7, 32, 48, 64, fpsk.BF16, 99, 3, 16, cache)
    assert lib.fpsk_bside_matches(C.byref(s), *args) == 0            # nothing cached yet
    s.B, s.cache, s.ldb, s.version, s.m, s.k, s.n = 0x1000, 0x2000, 64, 7, 32, 48, 64
    s.dtype, s.seed, s.round, s.n_buckets, s.valid = fpsk.BF16, 99, 3, 16, 1
    assert lib.fpsk_bside_matches(C.byref(s), *args) == 1
    for pos, other in ((0, C.c_void_p(0x1040)), (1, 128), (2, 8), (3, 33), (4, 49), (5, 65), (6, fpsk.FP16), (7, 98),
                       (8, 2), (9, 17), (10, C.c_void_p(0x3000))):
        changed = list(args)
        changed[pos] = other
        assert lib.fpsk_bside_matches(C.byref(s), *changed) == 0, pos   # any field of the key invalidates
    s.valid = 0
    assert lib.fpsk_bside_matches(C.byref(s), *args) == 0


def test_hashed_probe_validation_needs_no_device(lib):
    one = C.c_void_p(4096)
    s = fpsk.BSide()
    f = lib.fpsk_probe_hashed

    def call(side=s, A=one, c_is_fp32=1, nb=16, rnd=0, cache=one, cbytes=1 << 30, ws=one, wbytes=1 << 30, m=64):
        return f(C.byref(side) if side is not None else None, A, 64, one, 64, 0, one, 64, m, 64, 64, fpsk.FP16, c_is_fp32,
                 1, rnd, nb, None, cache, cbytes, ws, wbytes, None, one, None, None)

    assert call(c_is_fp32=0) == fpsk.ERR_DTYPE          # a narrowed C is rejected
    assert call(side=None) == fpsk.ERR_NULL
    assert call(A=None) == fpsk.ERR_NULL
    assert call(m=0) == fpsk.ERR_SHAPE
    assert call(nb=0) == fpsk.ERR_BUCKETS and call(nb=5000) == fpsk.ERR_BUCKETS and call(rnd=-1) == fpsk.ERR_BUCKETS
    assert call(cache=C.c_void_p(4096 + 8)) == fpsk.ERR_ALIGN
    assert call(cbytes=16) == fpsk.ERR_WORKSPACE and call(wbytes=16) == fpsk.ERR_WORKSPACE
    assert s.valid == 0 and s.rebuilds == 0
    assert lib.fpsk_probe_hashed_cache_bytes(0, 8, 8, 4) == 0
    assert lib.fpsk_probe_hashed_workspace_bytes(64, 64, 64, 16) >= 4 * (16 * 64 * 2 + 16 * 16)


def test_probe_state_layout_cadence_and_recalibration_match_the_oracle(lib):
    assert C.sizeof(fpsk.ProbeState) == 32 and fpsk.ProbeState.sigma_sum.offset == 16
    for calls in list(range(0, 40)) + [1023, 1024, 1025, 1040, 2048, 4096, 5000]:
        assert fpsk.recalibration_due(calls) == O.recalibration_due(calls), calls
    for (n1, n3) in ((4096, 4096), (2048, 11008), (16384, 512)):
        for m_cur in (16, 48, 100, 256, 1000):
            for sig in (1e-9, 3e-6, 7.3e-5, 1e-4, 2e-3, 1.0, float("nan"), 0.0, float("inf")):
                for rms in (1.0, 0.37, 12.0, 0.0):
                    assert fpsk.probe_recalibrate(n1, n3, sig, rms, m_cur) == O.recalibrate_probe(n1, n3, sig, rms, m_cur)
    mn, rb = C.c_int32(), C.c_int32()
    assert lib.fpsk_probe_recalibrate(0, 4, 1.0, 1.0, 16, None, C.byref(mn), C.byref(rb)) == fpsk.ERR_SHAPE
    assert lib.fpsk_probe_recalibrate(4, 4, 1.0, 1.0, 0, None, C.byref(mn), C.byref(rb)) == fpsk.ERR_BUCKETS
    assert lib.fpsk_probe_recalibrate(4, 4, 1.0, 1.0, 16, None, None, C.byref(rb)) == fpsk.ERR_NULL
    assert lib.fpsk_probe_state_reset(None, None) == fpsk.ERR_NULL
    assert lib.fpsk_probe_accumulate(None, None, None) == fpsk.ERR_NULL
