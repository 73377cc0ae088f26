"""Parity of the CUDA library (through its C ABI) with the float64 oracle.

Tolerances (normalised max error  max|a-b| / max|b|  per tensor; element-wise
relative error is meaningless where outputs cross zero):
    x, grad_y  <= 1e-4        grad_w <= 1e-3
    log-det    |a-b| <= 1e-5 * max(|b|, H*W*1e-3)
"""
import numpy as np
import pytest

from conftest import nmax_err
from paper_2410_14634_b200 import workloads

pytestmark = pytest.mark.gpu

TOL_X = 1e-4
TOL_GW = 1e-3

PATHS = {"auto": 0, "generic": 1, "warp": 2, "team": 3, "tensor": 4}


@pytest.fixture(scope="module")
def B():
    from paper_2410_14634_b200 import binding
    binding.lib()
    yield binding
    binding.invconv_set_path(0)


@pytest.fixture(scope="module")
def oracle():
    from oracle import api
    return api


def dev(a):
    import torch
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def run_or_skip(binding, path, fn, *args, **kw):
    """A forced family may decline a shape (skip); the automatic choice must serve every shape."""
    try:
        return fn(*args, **kw)
    except binding.InvConvError as e:
        if e.status == binding.UNSUPPORTED:
            if path == "auto":
                pytest.fail("the automatic dispatch returned UNSUPPORTED")
            pytest.skip("this kernel family does not serve the shape")
        raise


def check_all(binding, oracle, w, y, gx, path, tol_x=TOL_X, tol_gw=TOL_GW):
    """Forward, backward (on the GPU's own x and on the oracle's x), f, log-det."""
    import torch
    Bn, C, H, W = y.shape
    k = w.shape[2]
    binding.invconv_set_path(PATHS[path])
    try:
        wd, yd, gxd = dev(w), dev(y), dev(gx)
        x = run_or_skip(binding, path, binding.invconv_forward, yd, wd)
        gy, gw = run_or_skip(binding, path, binding.invconv_backward, gxd, x, wd)
        x_ref = oracle.invconv_forward(y, w)
        gy_ref, gw_ref = oracle.invconv_backward(gx, x_ref, w)
        # backward again from the oracle's x rounded to fp32 (separates forward from backward error)
        gy2, gw2 = binding.invconv_backward(gxd, dev(x_ref.astype(np.float32)), wd)
        yy = binding.masked_conv_forward(x, wd)
        ld = binding.invconv_logdet(wd, H, W)
        torch.cuda.synchronize()
        assert binding.invconv_get_status() == 0
    finally:
        binding.invconv_set_path(0)
    if Bn > 0:
        assert nmax_err(x.cpu().numpy(), x_ref) <= tol_x
        assert nmax_err(gy.cpu().numpy(), gy_ref) <= tol_x
        assert nmax_err(gy2.cpu().numpy(), gy_ref) <= tol_x
        assert nmax_err(yy.cpu().numpy(), y) <= tol_x                 # f(f^{-1}(y)) = y on the device
    assert nmax_err(gw.cpu().numpy(), gw_ref) <= tol_gw
    assert nmax_err(gw2.cpu().numpy(), gw_ref) <= tol_gw
    ctr = gw.cpu().numpy()[:, :, k - 1, k - 1]
    assert np.all(ctr[np.triu_indices(C, 1)] == 0.0)                  # outside the mask: exact zeros
    ld_ref = oracle.logdet(w, H, W)
    assert abs(float(ld.item()) - ld_ref) <= 1e-5 * max(abs(ld_ref), H * W * 1e-3)


# ------------------------------------------------------------------ the ten benchmark shapes, full size

@pytest.mark.parametrize("path", ["auto", "generic", "warp", "team", "tensor"])
@pytest.mark.parametrize("name", [s.name for s in workloads.SHAPES])
def test_benchmark_shapes_full_size(B, oracle, name, path):
    s, w, y, gx = workloads.make(name)
    if path == "generic" and s.C * s.k * s.k > 1300:
        pytest.skip("fallback kernel on the heaviest shapes is covered by the smaller cases")
    check_all(B, oracle, w, y, gx, path)


# ------------------------------------------------------------------ small, ragged and degenerate shapes

EDGE = [  # (B, C, H, W, k)
    (1, 1, 1, 1, 1), (2, 1, 1, 1, 3), (1, 2, 1, 5, 2), (1, 3, 6, 1, 3), (2, 2, 2, 2, 4),
    (3, 1, 3, 3, 3), (2, 3, 5, 4, 3), (1, 2, 7, 9, 5), (2, 1, 13, 17, 2), (1, 3, 31, 29, 3),
    (2, 1, 33, 30, 3), (1, 3, 35, 37, 5), (1, 4, 9, 11, 3), (1, 5, 6, 7, 3), (1, 7, 5, 5, 2),
    (2, 12, 5, 7, 3), (1, 16, 9, 9, 3), (1, 33, 4, 6, 3), (1, 24, 8, 8, 5), (1, 1, 40, 70, 7),
    (1, 2, 16, 16, 11), (1, 1, 65, 66, 3), (1, 3, 100, 20, 3), (5, 1, 28, 28, 3),
    (1, 3, 100, 200, 3), (2, 1, 250, 260, 5), (1, 2, 70, 500, 2),       # larger than shared memory: global-memory mode
    (1, 1, 250, 257, 3), (1, 2, 130, 301, 5), (1, 4, 96, 180, 2), (1, 3, 200, 160, 3),   # ... ragged widths (4-byte ring copies), ring too large
    (1, 2, 12, 12, 9), (2, 3, 20, 24, 9),                                 # the paper's ablation also runs k = 9
    # tensor-core family: every channel count it serves, k = 2..5, fewer rows than lanes, wide and narrow images,
    # batches that do not fill a group of images, several groups per cluster
    (9, 16, 16, 16, 3), (3, 32, 8, 8, 5), (17, 48, 16, 4, 2), (5, 64, 12, 16, 4), (1, 48, 16, 16, 5),
    (20, 16, 7, 12, 5), (2, 32, 16, 32, 3), (200, 16, 4, 4, 3), (33, 48, 2, 2, 3), (4, 64, 16, 16, 5),
    # dynamic shared memory of exactly 48 KB beside a kernel's static words (needs the opt-in all the same)
    (6, 2, 37, 39, 5), (3, 2, 160, 114, 5),
    # kernel transform: more than 4096 right-hand-side values per input channel, four row slots per lane, one channel
    (1, 96, 4, 4, 7), (1, 128, 3, 3, 7), (2, 128, 4, 4, 3), (1, 100, 4, 4, 2), (2, 5, 8, 8, 1), (1, 40, 6, 6, 9),
]


@pytest.mark.parametrize("path", ["auto", "generic", "warp", "team", "tensor"])
@pytest.mark.parametrize("shape", EDGE, ids=lambda s: "x".join(map(str, s)))
def test_edge_shapes(B, oracle, shape, path):
    Bn, C, H, W, k = shape
    w, y, gx = workloads.make_custom(100 + sum(shape), Bn, C, H, W, k, sigma=0.05 / np.sqrt(C))
    check_all(B, oracle, w, y, gx, path)


@pytest.mark.parametrize("shape", [(18, 1, 25, 32, 1), (18, 2, 25, 32, 1), (6, 4, 16, 16, 1), (9, 5, 8, 16, 3)], ids=lambda s: "x".join(map(str, s)))
def test_grad_w_of_few_channels_keeps_fp32_accuracy_under_cancellation(B, oracle, shape):
    """Few entries in grad_w, each a long sum with heavy cancellation (sum of |terms| about 100 times the sum):
    operands rounded to TF32 would show at 1e-3 of the entry, so these shapes must stay on fp32 multiply-adds."""
    import torch
    Bn, C, H, W, k = shape
    for seed in range(6):
        w, y, gx = workloads.make_custom(seed, Bn, C, H, W, k, sigma=0.05)
        x_ref = oracle.invconv_forward(y, w)
        _, gw_ref = oracle.invconv_backward(gx, x_ref, w)
        _, gw = B.invconv_backward(dev(gx), dev(x_ref.astype(np.float32)), dev(w))
        torch.cuda.synchronize()
        assert nmax_err(gw.cpu().numpy(), gw_ref) <= 2e-5, seed


GW_SEPARATE = [  # shapes for the pixel-parallel grad_w kernel: ragged widths, bands with and without halo rows,
    # more (image, band) items than CTAs, a single pixel, every (C, k) the few-channel family serves
    (1, 1, 1, 1, 2), (3, 1, 28, 28, 3), (2, 3, 32, 32, 3), (1, 3, 64, 64, 5), (2, 4, 9, 11, 5), (1, 2, 7, 9, 5),
    (170, 1, 8, 8, 3), (300, 2, 4, 4, 2), (1, 4, 40, 36, 3), (2, 3, 33, 30, 2), (1, 1, 130, 260, 5), (5, 4, 16, 16, 5),
]


@pytest.mark.parametrize("separate", ["0", "1"])
@pytest.mark.parametrize("shape", GW_SEPARATE, ids=lambda s: "x".join(map(str, s)))
def test_grad_w_inside_or_after_the_wavefront(B, oracle, shape, separate):
    """Both ways of computing grad_w on the few-channel path (riding along in the wavefront kernel, or the
    pixel-parallel kernel after it) against the oracle, and twice in a row (the ticket counter is reset)."""
    prev = B.invconv_set_option(B.OPT_GRADW_SEPARATE, int(separate))
    try:
        Bn, C, H, W, k = shape
        w, y, gx = workloads.make_custom(300 + sum(shape), Bn, C, H, W, k, sigma=0.05 / np.sqrt(C))
        check_all(B, oracle, w, y, gx, "warp")
        check_all(B, oracle, w, y, gx, "warp")
    finally:
        B.invconv_set_option(B.OPT_GRADW_SEPARATE, prev)


def test_grad_w_after_the_wavefront_with_unaligned_buffers(B, oracle):
    """Buffers that start 4 bytes off a 16-byte boundary take the plain-load staging path."""
    import torch
    prev = B.invconv_set_option(B.OPT_GRADW_SEPARATE, 1)
    Bn, C, H, W, k = 3, 3, 12, 16, 3
    w, y, gx = workloads.make_custom(77, Bn, C, H, W, k)
    n = y.size
    def off(a):
        buf = torch.empty(n + 1, dtype=torch.float32, device="cuda")
        v = buf[1:].view(a.shape)
        v.copy_(torch.from_numpy(a))
        return v
    B.invconv_set_path(PATHS["warp"])
    try:
        x = B.invconv_forward(off(y), dev(w))
        gy = torch.empty(n + 1, dtype=torch.float32, device="cuda")[1:].view(y.shape)
        _, gw = B.invconv_backward(off(gx), off(x.cpu().numpy()), dev(w), out_grad_y=gy)
        torch.cuda.synchronize()
        assert B.invconv_get_status() == 0
    finally:
        B.invconv_set_path(0)
        B.invconv_set_option(B.OPT_GRADW_SEPARATE, prev)
    x64 = x.cpu().numpy().astype(np.float64)
    gy_ref = oracle.invconv_grad_y(gx, w)
    gw_ref = oracle.invconv_grad_w(gy_ref, x64, w.shape[-1])
    assert nmax_err(gy.cpu().numpy(), gy_ref) <= 1e-4
    assert nmax_err(gw.cpu().numpy(), gw_ref) <= 1e-3


@pytest.mark.parametrize("path", ["auto", "generic", "warp", "team"])
def test_masked_out_kernel_entries_are_never_read(B, oracle, path):
    for (Bn, C, H, W, k) in [(2, 3, 9, 8, 3), (1, 12, 6, 6, 3)]:
        w, y, gx = workloads.make_custom(7, Bn, C, H, W, k, masked_fill=float("nan"))
        check_all(B, oracle, w, y, gx, path)


@pytest.mark.parametrize("path", ["auto", "generic", "warp", "team"])
def test_paper_setting_unit_diagonal_one_channel(B, oracle, path):
    """The paper's own assumption: one channel, bottom-right entry equal to 1; log-det is exactly 0."""
    w, y, gx = workloads.make_custom(8, 3, 1, 12, 10, 3, diag_lo=1.0, diag_hi=1.0)
    assert w[0, 0, 2, 2] == 1.0
    check_all(B, oracle, w, y, gx, path)
    assert float(B.invconv_logdet(dev(w), 12, 10).item()) == 0.0


@pytest.mark.parametrize("path", ["auto", "generic", "team"])
@pytest.mark.parametrize("shape", [(3, 1, 28, 28, 3), (2, 3, 32, 32, 3), (2, 3, 40, 45, 5), (1, 2, 7, 70, 2), (2, 4, 9, 9, 5),
                                   # few or large images: one CTA per band of rows (bands that do not divide the
                                   # height, a one-row last band, images larger than shared memory, widths off 4)
                                   (2, 3, 64, 64, 5), (1, 1, 256, 256, 5), (3, 2, 40, 36, 3), (1, 4, 100, 20, 2),
                                   (5, 1, 17, 8, 3), (1, 3, 65, 64, 3), (1, 1, 300, 260, 5), (2, 2, 33, 30, 3), (16, 3, 64, 64, 5),
                                   # tensor-core kernel ("auto" at C = 16..64; "team" keeps the FMA tile kernel): every k
                                   # it serves, bands that do not fill the lanes, ragged last band, wide and 1-pixel-high
                                   # images, more tiles than CTAs, the two 48-channel benchmark shapes
                                   (3, 16, 16, 16, 3), (2, 32, 9, 20, 5), (1, 48, 8, 8, 3), (2, 64, 12, 7, 4), (3, 16, 1, 100, 2),
                                   (170, 16, 4, 4, 3), (1, 48, 50, 30, 5), (64, 48, 16, 16, 5), (64, 48, 16, 16, 3),
                                   (2, 12, 16, 16, 3), (1, 3, 5, 5, 7),
                                   # many channels (register-tiled kernel): ragged widths, several bands per image,
                                   # several images per CTA, channel counts off the tile sizes, every k it serves
                                   (3, 5, 7, 9, 2), (2, 13, 20, 20, 4), (1, 33, 6, 10, 5), (1, 6, 40, 36, 3), (2, 7, 5, 5, 1),
                                   (5, 96, 8, 8, 5), (1, 8, 3, 250, 3), (1, 8, 3, 260, 3), (9, 17, 4, 4, 3), (2, 6, 9, 9, 7)],
                         ids=lambda s: "x".join(map(str, s)))
def test_masked_conv_matches_oracle(B, oracle, shape, path):
    """y = f(x) on its own (the sampling direction), junk in the masked-out kernel entries."""
    import torch
    Bn, C, H, W, k = shape
    w, x, _ = workloads.make_custom(31 + sum(shape), Bn, C, H, W, k, sigma=0.3 / np.sqrt(C), masked_fill=float("nan"))
    B.invconv_set_path(PATHS[path])
    try:
        y = B.masked_conv_forward(dev(x), dev(w))
        torch.cuda.synchronize()
    finally:
        B.invconv_set_path(0)
    assert nmax_err(y.cpu().numpy(), oracle.masked_conv(x, w)) <= 1e-5


@pytest.mark.parametrize("shape", [(4, 3, 16, 16, 3), (3, 1, 28, 28, 3), (2, 12, 8, 8, 3), (2, 5, 6, 7, 2),
                                   (2, 3, 64, 64, 5), (1, 1, 250, 257, 3), (9, 48, 16, 16, 3), (3, 96, 8, 8, 3), (1, 3, 8, 8, 7)],
                         ids=lambda s: "x".join(map(str, s)))
def test_training_step_calls_with_the_log_det_folded_in(B, oracle, shape):
    """invconv_forward_logdet / invconv_backward_logdet against the oracle's x, logdet, grad_y and
    grad_w + grad_logdet * d logdet / d w, for every place the log-det is emitted from (the warp kernel, the
    separate grad_w kernel of large images, the kernel transform and grad_w reductions of the team and tensor
    families, the fallback kernels)."""
    import torch
    Bn, C, H, W, k = shape
    w, y, gx = workloads.make_custom(500 + sum(shape), Bn, C, H, W, k, sigma=0.05 / np.sqrt(C))
    gl = -0.37
    x, ld = B.invconv_forward_logdet(dev(y), dev(w))
    gy, gw = B.invconv_backward_logdet(dev(gx), x, dev(w), torch.tensor([gl], dtype=torch.float32, device="cuda"))
    torch.cuda.synchronize()
    assert B.invconv_get_status() == 0
    x_ref = oracle.invconv_forward(y, w)
    gy_ref, gw_ref = oracle.invconv_backward(gx, x_ref, w)
    gw_ref = gw_ref + gl * oracle.logdet_grad_w(w, H, W)
    ld_ref = oracle.logdet(w, H, W)
    assert nmax_err(x.cpu().numpy(), x_ref) <= TOL_X
    assert nmax_err(gy.cpu().numpy(), gy_ref) <= TOL_X
    assert nmax_err(gw.cpu().numpy(), gw_ref) <= TOL_GW
    assert abs(float(ld.item()) - ld_ref) <= 1e-5 * max(abs(ld_ref), H * W * 1e-3)
    # the diagonal term alone, where it dominates: compare the difference to plain backward
    _, gw0 = B.invconv_backward(dev(gx), x, dev(w))
    d = (gw - gw0).cpu().numpy().astype(np.float64)
    assert nmax_err(d, gl * oracle.logdet_grad_w(w, H, W)) <= 1e-5


@pytest.mark.parametrize("mma", [0, 1])
@pytest.mark.parametrize("family", ["team", "tensor"])
@pytest.mark.parametrize("shape", [(3, 48, 8, 8, 3), (2, 40, 6, 16, 2), (2, 33, 16, 16, 5), (5, 96, 8, 8, 3), (2, 40, 8, 8, 5),
                                   (5, 64, 16, 16, 5), (4, 32, 12, 16, 4), (64, 48, 16, 16, 5), (64, 96, 8, 8, 3)],
                         ids=lambda s: "x".join(map(str, s)))
def test_grad_w_many_channels_fma_and_tensor_pipe(B, oracle, shape, mma, family):
    """grad_w at many channels through the fp32 FMA kernel and through the tensor-pipe kernels (tf32 operands;
    mma.sync in the team family, tcgen05 in the tensor family), channel counts on and off the tile size, k up
    to 5, the two widest benchmark shapes at full size.  Both stay inside the 1e-3 bar (normalised by the
    largest entry); the FMA kernel, which keeps fp32 inputs, far inside it.  For the tensor pipe the
    element-wise relative error is checked too, on the entries that carry weight (at least a tenth of the
    largest): tf32 operands give every entry an error of about 3e-4 of the LARGEST entry."""
    prev = B.invconv_set_option(B.OPT_GRADW_TENSOR_PIPE, mma)
    Bn, C, H, W, k = shape
    w, y, gx = workloads.make_custom(700 + sum(shape), Bn, C, H, W, k, sigma=0.05 / np.sqrt(C))
    x_ref = oracle.invconv_forward(y, w)
    gy_ref, gw_ref = oracle.invconv_backward(gx, x_ref, w)
    B.invconv_set_path(PATHS[family])
    try:
        _, gw = run_or_skip(B, "forced", B.invconv_backward, dev(gx), dev(x_ref.astype(np.float32)), dev(w))
    finally:
        B.invconv_set_path(0)
        B.invconv_set_option(B.OPT_GRADW_TENSOR_PIPE, prev)
    g = gw.cpu().numpy().astype(np.float64)
    err = nmax_err(g, gw_ref)
    assert err <= (TOL_GW if mma == 1 else 2e-5), err
    big = np.abs(gw_ref) >= 0.1 * np.abs(gw_ref).max()
    rel = np.max(np.abs(g - gw_ref)[big] / np.abs(gw_ref)[big])
    assert rel <= (5e-3 if mma == 1 else 2e-4), rel


@pytest.mark.parametrize("name", ["mnist", "cifar_sq", "wide48_k3"])
def test_batch_shards_sum_to_the_full_grad_w(B, oracle, name):
    """The multi-GPU partition on one GPU: images are independent and grad_w is a sum over the batch, so two
    half-batches run one after the other give the full batch's x and grad_y and, summed, its grad_w (what the
    all-reduce does across ranks)."""
    import torch
    from paper_2410_14634_b200 import sharding
    s, w, y, gx = workloads.make(name)
    wd = dev(w)
    xs, gys, gw_sum = [], [], None
    for rank in range(2):
        start, count = sharding.shard_batch(s.B, 2, rank)
        x = B.invconv_forward(dev(y[start:start + count]), wd)
        gy, gw = B.invconv_backward(dev(gx[start:start + count]), x, wd)
        xs.append(x); gys.append(gy)
        gw_sum = gw.clone() if gw_sum is None else gw_sum + gw
    torch.cuda.synchronize()
    x_ref = oracle.invconv_forward(y, w)
    gy_ref, gw_ref = oracle.invconv_backward(gx, x_ref, w)
    assert nmax_err(torch.cat(xs).cpu().numpy(), x_ref) <= TOL_X
    assert nmax_err(torch.cat(gys).cpu().numpy(), gy_ref) <= TOL_X
    assert nmax_err(gw_sum.cpu().numpy(), gw_ref) <= TOL_GW


def test_a_bounded_wait_that_runs_out_is_reported_once_and_the_context_stays_usable(B, oracle):
    """The failure path of the device-side waits, without a fault: a probe kernel waits on a barrier that
    nothing completes, gives up after its limit, raises the status word and returns.  The status query reports
    INVCONV_TIMEOUT exactly once, and the next forward call is still correct."""
    import torch
    assert B.invconv_get_status() == 0
    B.invconv_selftest_wait_timeout(20000)
    torch.cuda.synchronize()
    assert B.invconv_get_status() == B.TIMEOUT
    assert B.invconv_get_status() == 0
    s, w, y, gx = workloads.make("pr1")
    x = B.invconv_forward(dev(y), dev(w))
    torch.cuda.synchronize()
    assert B.invconv_get_status() == 0
    assert nmax_err(x.cpu().numpy(), oracle.invconv_forward(y, w)) <= TOL_X


@pytest.mark.parametrize("shape", [(3, 16, 8, 8, 3), (9, 48, 16, 16, 3), (3, 64, 16, 24, 3), (7, 64, 15, 24, 2)], ids=lambda s: "x".join(map(str, s)))
def test_unaligned_buffers_on_shapes_of_the_tensor_family(B, oracle, shape):
    """Buffers 4 bytes off a 16-byte boundary: the automatic choice must still serve the shape (the tensor family's
    bulk copies need aligned slices, so another family takes over), forward, backward and masked convolution."""
    import torch
    Bn, C, H, W, k = shape
    w, y, gx = workloads.make_custom(55 + sum(shape), Bn, C, H, W, k, sigma=0.05 / np.sqrt(C))

    def off(a):
        buf = torch.empty(a.size + 1, dtype=torch.float32, device="cuda")
        v = buf[1:].view(a.shape)
        v.copy_(torch.from_numpy(a))
        return v

    n = y.size
    x = torch.empty(n + 1, dtype=torch.float32, device="cuda")[1:].view(y.shape)
    gy = torch.empty(n + 1, dtype=torch.float32, device="cuda")[1:].view(y.shape)
    yy = torch.empty(n + 1, dtype=torch.float32, device="cuda")[1:].view(y.shape)
    B.invconv_forward(off(y), dev(w), out=x)
    _, gw = B.invconv_backward(off(gx), x, dev(w), out_grad_y=gy)
    B.masked_conv_forward(x, dev(w), out=yy)
    torch.cuda.synchronize()
    assert B.invconv_get_status() == 0
    x_ref = oracle.invconv_forward(y, w)
    gy_ref, gw_ref = oracle.invconv_backward(gx, x_ref, w)
    assert nmax_err(x.cpu().numpy(), x_ref) <= TOL_X and nmax_err(gy.cpu().numpy(), gy_ref) <= TOL_X
    assert nmax_err(gw.cpu().numpy(), gw_ref) <= TOL_GW and nmax_err(yy.cpu().numpy(), y) <= TOL_X


def test_empty_batch_is_a_no_op_and_zeroes_grad_w(B):
    import torch
    w = dev(workloads.make_custom(9, 1, 2, 4, 4, 3)[0])
    y = torch.empty(0, 2, 4, 4, device="cuda")
    x = B.invconv_forward(y, w)
    gy, gw = B.invconv_backward(y, x, w)
    torch.cuda.synchronize()
    assert x.shape == y.shape and gy.shape == y.shape
    assert torch.all(gw == 0)


def test_results_are_bitwise_reproducible(B):
    import torch
    for name in ("pr1", "cifar_sq"):
        s, w, y, gx = workloads.make(name)
        wd, yd, gxd = dev(w), dev(y), dev(gx)
        x1 = B.invconv_forward(yd, wd)
        gy1, gw1 = B.invconv_backward(gxd, x1, wd)
        x2 = B.invconv_forward(yd, wd)
        gy2, gw2 = B.invconv_backward(gxd, x2, wd)
        torch.cuda.synchronize()
        assert torch.equal(x1, x2) and torch.equal(gy1, gy2) and torch.equal(gw1, gw2)


def test_plain_entry_points_match_workspace_entry_points(B):
    """invconv_forward / invconv_backward (library-managed scratch) against the _ws forms the binding uses."""
    import torch
    for name in ("pr1", "cifar_sq"):
        s, w, y, gx = workloads.make(name)
        wd, yd, gxd = dev(w), dev(y), dev(gx)
        x_ws = B.invconv_forward(yd, wd)
        gy_ws, gw_ws = B.invconv_backward(gxd, x_ws, wd)
        x = torch.empty_like(yd); gy = torch.empty_like(yd); gw = torch.empty_like(wd)
        L = B.lib()
        st = torch.cuda.current_stream().cuda_stream
        assert L.invconv_forward(yd.data_ptr(), wd.data_ptr(), x.data_ptr(), s.B, s.C, s.H, s.W, s.k, st) == 0
        assert L.invconv_backward(gxd.data_ptr(), x.data_ptr(), wd.data_ptr(), gy.data_ptr(), gw.data_ptr(),
                                  s.B, s.C, s.H, s.W, s.k, st) == 0
        torch.cuda.synchronize()
        assert torch.equal(x, x_ws) and torch.equal(gy, gy_ws) and torch.equal(gw, gw_ws)


def test_grad_w_may_be_skipped(B):
    import torch
    s, w, y, gx = workloads.make("pr1")
    wd, yd, gxd = dev(w), dev(y), dev(gx)
    x = B.invconv_forward(yd, wd)
    gy_a, _ = B.invconv_backward(gxd, x, wd)
    gy_b, none = B.invconv_backward(gxd, x, wd, need_grad_w=False)
    torch.cuda.synchronize()
    assert none is None and torch.equal(gy_a, gy_b)


def test_host_step_matches_oracle(B, oracle):
    import torch
    s, w, y, gx = workloads.make("pr1")
    hs = B.HostStep(s.B, s.C, s.H, s.W, s.k)
    hs.y.copy_(torch.from_numpy(y)); hs.w.copy_(torch.from_numpy(w)); hs.grad_x.copy_(torch.from_numpy(gx))
    for _ in range(2):
        hs.run()
        torch.cuda.synchronize()
        x_ref = oracle.invconv_forward(y, w)
        gy_ref, gw_ref = oracle.invconv_backward(gx, x_ref, w)
        assert nmax_err(hs.x.numpy(), x_ref) <= TOL_X
        assert nmax_err(hs.grad_y.numpy(), gy_ref) <= TOL_X
        assert nmax_err(hs.grad_w.numpy(), gw_ref) <= TOL_GW
        ld_ref = oracle.logdet(w, s.H, s.W)
        assert abs(float(hs.logdet.item()) - ld_ref) <= 1e-5 * max(abs(ld_ref), s.H * s.W * 1e-3)


def test_bad_arguments_return_status_codes(B):
    import torch
    L = B.lib()
    t = torch.zeros(64, device="cuda")
    p = t.data_ptr()
    assert L.invconv_forward(p, p, p, 1, 1, 4, 4, 3, None) == B.BAD_ARG            # x aliases y
    assert L.invconv_forward(None, p, p, 1, 1, 4, 4, 3, None) == B.BAD_ARG
    assert L.invconv_backward(p, p, p, None, None, 1, 1, 4, 4, 3, None) == B.BAD_ARG
    assert L.invconv_forward(p, p, p, 1, 1, 4, 4, 12, None) == B.UNSUPPORTED
    assert L.masked_conv_forward(p, p, p, 1, 1, 4, 4, 3, None) == B.BAD_ARG
    assert B.invconv_get_status() == 0


def test_step_latency_probes_run(B):
    for mech in (0, 1, 2):
        c = B.invconv_probe_step_latency(mech, 2048)
        assert 1.0 < c < 5000.0
