"""Harness pieces shared by the GPU tests, the smoke check and the benchmark: the vendor
FP32-output GEMM under test and a few timing helpers.  None of this is part of the verifier."""
from __future__ import annotations

import torch


def vendor_gemm_fp32(A: torch.Tensor, B: torch.Tensor) -> torch.Tensor:
    """The unmodified vendor GEMM under test: half-precision operands on the tensor cores,
    FP32 accumulator delivered un-narrowed (cuBLASLt compute type 32F with an FP32 result)."""
    assert A.is_cuda and B.is_cuda
    return torch.mm(A, B, out_dtype=torch.float32)


def time_cuda(fn, iters: int, stream=None):
    """Median and mean per-call milliseconds of fn() over `iters` calls, CUDA events on the
    current stream, one synchronisation at each end."""
    evs = [torch.cuda.Event(enable_timing=True) for _ in range(iters + 1)]
    torch.cuda.synchronize()
    evs[0].record()
    for i in range(iters):
        fn(i)
        evs[i + 1].record()
    torch.cuda.synchronize()
    ts = sorted(evs[i].elapsed_time(evs[i + 1]) for i in range(iters))
    total = evs[0].elapsed_time(evs[iters])
    return ts[len(ts) // 2], total / iters, ts
