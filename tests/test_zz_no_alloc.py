"""The allocation-free GEMM entry point (collected last on purpose).

wd_op_gemm_noalloc serves callers that cannot allocate scratch memory where they
call from (code inside another framework's memory pool, loops that ban allocator
calls once running).  It keeps its split-K partial sums in a fixed array inside
the library, shared by all calls, so the checks here are: it agrees with the
ordinary entry point and with the float64 product of the same operands, also on a
second call that finds the first call's leftovers in the array, and it refuses
shapes the array cannot hold."""
import gc

import numpy as np
import pytest
import torch

from paper_2601_20332_b200 import binding as wd
from paper_2601_20332_b200 import build as wd_build

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _pair(rows, n, k, seed):
    g = torch.Generator(device=DEV).manual_seed(seed)
    x = torch.randn(rows, k, device=DEV, generator=g).to(torch.bfloat16)
    w = (torch.randn(n, k, device=DEV, generator=g) * 0.05).to(torch.bfloat16)
    return x, w


def test_noalloc_gemm_matches_ordinary_entry_point_twice_in_a_row():
    wd_build.build()
    # first call: several K slices fill a large part of the fixed array
    x1, w1 = _pair(34, 12288, 4096, 1)
    y1 = torch.empty(34, 12288, dtype=torch.float32, device=DEV)
    ref1 = wd.op_gemm(x1, w1, wd.WD_GEMM_TCGEN05)
    # second call: a different, smaller shape whose slices overlap the leftovers of the first
    x2, w2 = _pair(7, 1000, 264, 2)
    y2 = torch.empty(7, 1000, dtype=torch.float32, device=DEV)
    ref2 = wd.op_gemm(x2, w2, wd.WD_GEMM_TCGEN05)
    gc.collect()                       # tensors of earlier tests must not be freed between the two readings
    torch.cuda.synchronize()
    before = torch.cuda.memory_allocated()
    wd.op_gemm_noalloc(x1, w1, y1)
    wd.op_gemm_noalloc(x2, w2, y2)
    torch.cuda.synchronize()
    assert torch.cuda.memory_allocated() == before
    assert wd.op_status() == 0
    for y, ref, (x, w) in ((y1, ref1, (x1, w1)), (y2, ref2, (x2, w2))):
        a, b = y.cpu().numpy().astype(np.float64), ref.cpu().numpy().astype(np.float64)
        assert np.isfinite(a).all()
        assert np.abs(a - b).max() / np.abs(b).max() < 2e-5
        # and against the definition itself: the float64 product of the same bf16 operands
        exact = x.double().cpu().numpy() @ w.double().cpu().numpy().T
        assert np.abs(a - exact).max() / np.abs(exact).max() < 2e-5
    # and the first shape once more, now over the second call's leftovers
    y3 = torch.empty_like(y1)
    wd.op_gemm_noalloc(x1, w1, y3)
    torch.cuda.synchronize()
    assert np.abs(y3.cpu().numpy() - ref1.cpu().numpy()).max() / np.abs(ref1.cpu().numpy()).max() < 2e-5


def test_noalloc_gemm_rejects_what_the_fixed_array_cannot_hold():
    wd_build.build()
    L = wd.lib()
    cap = L.wd_op_gemm_noalloc_max_floats()
    assert cap == 4 << 20
    rows, n = 64, cap // 64 + 128                      # rows * n just above the limit
    x = torch.zeros(rows, 64, dtype=torch.bfloat16, device=DEV)
    w = torch.zeros(n, 64, dtype=torch.bfloat16, device=DEV)
    y = torch.zeros(rows, n, dtype=torch.float32, device=DEV)
    assert L.wd_op_gemm_noalloc(x.data_ptr(), w.data_ptr(), y.data_ptr(), rows, n, 64, None) == wd.WD_ERR_CAPACITY
    assert L.wd_op_gemm_noalloc(None, w.data_ptr(), y.data_ptr(), rows, n, 64, None) == wd.WD_ERR_NULL
    assert L.wd_op_gemm_noalloc(x.data_ptr(), w.data_ptr(), y.data_ptr(), rows, 128, 60, None) == wd.WD_ERR_BAD_PARAM
    # exactly at the limit is accepted
    n_ok = cap // 64
    assert L.wd_op_gemm_noalloc(x.data_ptr(), w.data_ptr(), y.data_ptr(), rows, n_ok, 64, None) == wd.WD_OK
    torch.cuda.synchronize()
    assert wd.op_status() == 0
