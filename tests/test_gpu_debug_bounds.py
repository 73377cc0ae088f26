"""The debug-bounds build (checked accessors in the tensor-core and flow-step kernels; the stand-in for a memory
checker on this pool): the accessor records an out-of-range index it is handed on purpose -- no memory is touched
-- and small, ragged and full-size cases of every kernel it covers run without a single recorded violation and
with the usual parity."""
import numpy as np
import pytest

from conftest import nmax_err
from paper_2410_14634_b200 import workloads

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def dbg():
    """The binding bound to libinvconv_b200_debug.so (built on demand); the regular library is restored afterwards."""
    from paper_2410_14634_b200 import binding, build
    path = build.build_debug_bounds()
    saved = (binding._lib, binding.LIB_PATH)
    binding._lib, binding.LIB_PATH = None, path
    binding.lib()
    yield binding
    binding._lib, binding.LIB_PATH = saved


def dev(a):
    import torch
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).cuda()


def test_the_accessor_records_a_bad_index_and_the_status_reports_it(dbg):
    import torch
    assert dbg.invconv_get_status() == 0
    assert dbg.lib().invconv_selftest_bounds(None) == dbg.OK
    torch.cuda.synchronize()
    assert dbg.invconv_get_status() == dbg.BOUNDS
    site, index, limit, count = dbg.invconv_debug_bounds_info()
    assert (site, index, limit, count) == (999, 5, 3, 1)
    assert dbg.invconv_debug_bounds_info() == (0, 0, 0, 0)          # the record is cleared by the query
    assert dbg.invconv_get_status() == 0


@pytest.mark.parametrize("shape", [(9, 16, 16, 16, 3), (3, 32, 8, 8, 5), (17, 48, 16, 4, 2), (5, 64, 12, 16, 4), (20, 16, 7, 12, 5),
                                   (33, 48, 2, 2, 3), (64, 48, 16, 16, 5), (3, 96, 8, 8, 3), (2, 32, 9, 20, 5), (3, 16, 1, 100, 2)],
                         ids=lambda s: "x".join(map(str, s)))
def test_no_violation_on_the_shapes_the_checked_kernels_serve(dbg, shape):
    import torch
    from oracle import api as oracle, flow_step
    Bn, C, H, W, k = shape
    w, y, gx = workloads.make_custom(900 + sum(shape), Bn, C, H, W, k, sigma=0.05 / np.sqrt(C))
    rng = np.random.default_rng(1)
    s, b = rng.uniform(0.5, 1.5, C).astype(np.float32), rng.normal(0, 0.3, C).astype(np.float32)
    V = (np.linalg.qr(rng.normal(size=(C, C)))[0]).astype(np.float32)
    wd = dev(w)
    x = dbg.invconv_forward(dev(y), wd)
    gy, gw = dbg.invconv_backward(dev(gx), x, wd)
    yy = dbg.masked_conv_forward(x, wd)
    x2, u, ld = dbg.invconv_flow_step_forward(dev(y), wd, dev(s), dev(b), dev(V))
    torch.cuda.synchronize()
    assert dbg.invconv_get_status() == 0
    assert dbg.invconv_debug_bounds_info() == (0, 0, 0, 0)
    x_ref = oracle.invconv_forward(y, w)
    gy_ref, gw_ref = oracle.invconv_backward(gx, x_ref, w)
    assert nmax_err(x.cpu().numpy(), x_ref) <= 1e-4 and nmax_err(gy.cpu().numpy(), gy_ref) <= 1e-4
    assert nmax_err(gw.cpu().numpy(), gw_ref) <= 1e-3 and nmax_err(yy.cpu().numpy(), y) <= 1e-4
    assert nmax_err(u.cpu().numpy(), flow_step.step_forward(y, w, s, b, V)[1]) <= 1e-4
