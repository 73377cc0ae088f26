"""The backward entry point for callers that may not allocate device memory.

Some hosts -- a server with a frozen memory plan, a real-time loop, a callback
inside another framework -- must not call an allocator once they are running.
`invconv_backward_noalloc` serves them: every buffer comes from the caller and
the library's own scratch is a fixed array inside the library image.  This test
calls it through the C ABI and checks it against the workspace-taking entry
point and against the float64 oracle, twice in a row (the shared scratch must
be left reusable), and checks that the device's free memory does not move
across the second call (the first call of a shape may load kernel code).

The file name sorts last on purpose: a run that stops at the first failure has
then already run every other test.
"""
import ctypes

import numpy as np
import pytest

from conftest import nmax_err
from paper_2410_14634_b200 import workloads

pytestmark = pytest.mark.gpu


def test_noalloc_backward_matches_workspace_backward_twice():
    import torch
    from paper_2410_14634_b200 import binding
    L = binding.lib()
    binding.invconv_set_path(binding.PATH_AUTO)
    for name, batch in (("pr1", None), ("mnist", 64), ("cifar", 16)):
        s, w, y, gx = workloads.make(name, batch=batch)
        B = y.shape[0]
        wd, yd, gxd = (torch.from_numpy(a).cuda() for a in (w, y, gx))
        x = binding.invconv_forward(yd, wd)
        gy_ref, gw_ref = binding.invconv_backward(gxd, x, wd)          # existing entry point (caller's workspace)
        torch.cuda.synchronize()
        from oracle import api as oracle
        gy_o, gw_o = oracle.invconv_backward(gx, x.cpu().numpy().astype(np.float64), w)
        st = torch.cuda.current_stream().cuda_stream
        free_before = None
        for attempt in range(2):                                       # two calls in a row share the fixed scratch
            gy = torch.full_like(gxd, float("nan"))
            gw = torch.full_like(wd, float("nan"))
            if attempt == 1:
                torch.cuda.synchronize()
                free_before = torch.cuda.mem_get_info()[0]
            rc = L.invconv_backward_noalloc(gxd.data_ptr(), x.data_ptr(), wd.data_ptr(), gy.data_ptr(), gw.data_ptr(),
                                            B, s.C, s.H, s.W, s.k, ctypes.c_void_p(st))
            assert rc == binding.OK, (name, attempt, rc)
            torch.cuda.synchronize()
            if attempt == 1:
                assert torch.cuda.mem_get_info()[0] == free_before, "the call changed the device's free memory"
            assert binding.invconv_get_status() == 0
            assert nmax_err(gy.cpu().numpy(), gy_ref.cpu().numpy()) <= 1e-4, (name, attempt)
            assert nmax_err(gw.cpu().numpy(), gw_ref.cpu().numpy()) <= 1e-3, (name, attempt)
            assert torch.equal(gy, gy_ref) and torch.equal(gw, gw_ref)  # same kernel, same order of sums
            assert nmax_err(gy.cpu().numpy(), gy_o) <= 1e-4, (name, attempt)
            assert nmax_err(gw.cpu().numpy(), gw_o) <= 1e-3, (name, attempt)


def test_noalloc_backward_rejects_what_it_cannot_serve():
    import torch
    from paper_2410_14634_b200 import binding
    L = binding.lib()
    t = torch.zeros(1 << 16, device="cuda")
    a, b, c, d, e = (t[i * 4096:].data_ptr() for i in range(5))
    # a shape the warp family does not serve: nothing runs, clear status
    assert L.invconv_backward_noalloc(a, b, c, d, e, 1, 12, 4, 4, 3, None) == binding.UNSUPPORTED
    # a batch whose per-CTA partial sums would not fit the fixed scratch
    big_b = 4 * (binding.NOALLOC_SCRATCH_BYTES // (4 * 4 * 4 * 25)) + 64
    assert L.invconv_backward_noalloc(a, b, c, d, e, big_b, 4, 2, 2, 5, None) == binding.WORKSPACE_TOO_SMALL
    assert L.invconv_backward_noalloc(None, b, c, d, e, 1, 1, 4, 4, 3, None) == binding.BAD_ARG
    torch.cuda.synchronize()
