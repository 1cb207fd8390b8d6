"""The allocation-free projection entry point, for hosts that cannot call cudaMalloc while running
(a process whose device memory all belongs to its own arena, or a loop that may not block or fail on
an allocation).  It must give what the context-based entry point gives, call after call, although
all calls share one fixed scratch array that still holds the previous call's partial sums.

Collected last on purpose: a run that stops at the first failure has then run every other test.
"""
import gc

import numpy as np
import pytest
import torch

from paper_2510_04147_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def test_noalloc_gemm_matches_context_gemm_twice_in_a_row():
    from paper_2510_04147_b200 import binding as b
    ssd = b.Ssd(b.config_from_workload(wl.TINY, max_drafts=4, max_batch=3))
    try:
        # two different problems back to back: the second must not see the first one's leftovers
        for call, (rows, n, k, split) in enumerate([(96, 1024, 2048, 4), (37, 640, 520, 3)]):
            x = wl.normal_tensor(21 + call, 1, (rows, k), 1.0, device="cuda", dtype=torch.bfloat16)
            w = wl.normal_tensor(21 + call, 2, (n, k), 0.05, device="cuda", dtype=torch.bfloat16)
            out = torch.full((rows, n), float("nan"), dtype=torch.float32, device="cuda")
            if call == 0:
                # the first call on a device looks up the array (and may make the driver load the kernels' module):
                # allowed to take device memory once, before the calls that must not
                assert b.gemm_bf16_noalloc(x, w, out, split) == 0
                out.fill_(float("nan"))
            # (tensors of earlier tests that only a collection frees must not be freed in the middle of the comparison)
            gc.collect()
            torch.cuda.synchronize()
            gc.disable()
            try:
                before, free_before = torch.cuda.memory_allocated(), torch.cuda.mem_get_info()[0]
                rc = b.gemm_bf16_noalloc(x, w, out, split)
                torch.cuda.synchronize()
                after, free_after = torch.cuda.memory_allocated(), torch.cuda.mem_get_info()[0]
            finally:
                gc.enable()
            assert rc == 0
            assert after == before
            assert free_after == free_before      # the driver handed out nothing either
            want = ssd.gemm_bf16(x, w, split)
            got, ref = out.cpu().numpy(), want.cpu().numpy()
            scale = np.sqrt(k) * 0.05
            tol = 2e-5 * scale * np.sqrt(k) + 1e-6           # the tolerance of the projection tests
            assert np.isfinite(got).all()
            assert np.abs(got - ref).max() <= tol
            exact = x.cpu().to(torch.float64).numpy() @ w.cpu().to(torch.float64).numpy().T
            assert np.abs(got - exact).max() < tol
    finally:
        ssd.destroy()


def test_noalloc_gemm_rejects_what_does_not_fit():
    from paper_2510_04147_b200 import binding as b
    x = torch.zeros((256, 64), dtype=torch.bfloat16, device="cuda")
    w = torch.zeros((4096, 64), dtype=torch.bfloat16, device="cuda")
    out = torch.zeros((256, 4096), dtype=torch.float32, device="cuda")
    assert b.gemm_bf16_noalloc(x, w, out, 1) == -5           # 256*4096 floats exceed the 4 MiB array: SSD_ERR_OVERFLOW
    assert b.gemm_bf16_noalloc(x[:128], w, out[:128], 1) == 0
    assert b.gemm_bf16_noalloc(x[:128], w, out[:128], 3) == -5
    assert b.gemm_bf16_noalloc(x[:128], w, out[:128], 9) == -2  # split_k outside [1, 8]: SSD_ERR_SHAPE
