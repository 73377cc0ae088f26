"""Parity of the flow-step calls (inverse convolution with Actnorm and the 1x1 convolution folded in; Section 4)
with the float64 oracle, through the C ABI: shapes served inside the warp-family kernel (one warp, several
warps, the channel-split walk), shapes composed from separate kernels (images in global memory, the team,
tensor and generic families), an empty batch."""
import numpy as np
import pytest

from conftest import nmax_err
from paper_2410_14634_b200 import workloads

pytestmark = pytest.mark.gpu

SHAPES = [(4, 3, 16, 16, 3), (5, 1, 28, 28, 3), (2, 4, 9, 11, 5), (3, 2, 33, 30, 3), (2, 3, 64, 64, 5), (7, 3, 32, 32, 3),
          (1, 1, 250, 257, 3), (2, 12, 16, 16, 3), (9, 48, 16, 16, 3), (1, 5, 6, 7, 3), (3, 96, 8, 8, 3), (1, 2, 1, 1, 1)]


def dev(a):
    import torch
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).cuda()


def neighbours(seed, C):
    rng = np.random.default_rng(seed)
    s = (rng.uniform(0.5, 1.5, size=C) * rng.choice([-1.0, 1.0], size=C)).astype(np.float32)
    b = rng.normal(0.0, 0.3, size=C).astype(np.float32)
    V = (np.linalg.qr(rng.normal(size=(C, C)))[0] + 0.1 * rng.normal(size=(C, C))).astype(np.float32)
    return s, b, V


@pytest.mark.parametrize("shape", SHAPES, ids=lambda s: "x".join(map(str, s)))
def test_flow_step_matches_oracle(shape):
    import torch
    from paper_2410_14634_b200 import binding
    from oracle import flow_step
    Bn, C, H, W, k = shape
    w, y, gu = workloads.make_custom(500 + sum(shape), Bn, C, H, W, k, sigma=0.05 / np.sqrt(C))
    s, b, V = neighbours(sum(shape), C)
    x_ref, u_ref, ld_ref = flow_step.step_forward(y, w, s, b, V)
    gy_ref, gw_ref, gs_ref, gb_ref, gV_ref = flow_step.step_backward(gu, x_ref, w, s, b, V)
    wd, sd, bd, Vd = dev(w), dev(s), dev(b), dev(V)
    for _ in range(2):                       # twice: scratch and control words are left reusable
        x, u, ld = binding.invconv_flow_step_forward(dev(y), wd, sd, bd, Vd)
        gy, gw, gs, gb, gV = binding.invconv_flow_step_backward(dev(gu), x, wd, sd, bd, Vd)
        torch.cuda.synchronize()
        assert binding.invconv_get_status() == 0
        assert nmax_err(x.cpu().numpy(), x_ref) <= 1e-4
        assert nmax_err(u.cpu().numpy(), u_ref) <= 1e-4
        assert abs(float(ld.item()) - ld_ref) <= 1e-5 * max(abs(ld_ref), H * W * 1e-3)
        assert nmax_err(gy.cpu().numpy(), gy_ref) <= 1e-4
        assert nmax_err(gw.cpu().numpy(), gw_ref) <= 1e-3
        assert nmax_err(gs.cpu().numpy(), gs_ref) <= 1e-4
        assert nmax_err(gb.cpu().numpy(), gb_ref) <= 1e-4
        assert nmax_err(gV.cpu().numpy(), gV_ref) <= 1e-4


def test_identity_neighbours_give_the_plain_layer_bit_for_bit():
    """s = 1, b = 0, V = I: u equals x exactly and the gradients equal those of invconv_backward."""
    import torch
    from paper_2410_14634_b200 import binding
    for shape in [(4, 3, 16, 16, 3), (2, 12, 16, 16, 3)]:
        Bn, C, H, W, k = shape
        w, y, gu = workloads.make_custom(41, Bn, C, H, W, k, sigma=0.05 / np.sqrt(C))
        wd = dev(w)
        s, b, V = dev(np.ones(C)), dev(np.zeros(C)), dev(np.eye(C))
        x, u, _ = binding.invconv_flow_step_forward(dev(y), wd, s, b, V)
        x0 = binding.invconv_forward(dev(y), wd)
        gy, gw, gs, gb, gV = binding.invconv_flow_step_backward(dev(gu), x, wd, s, b, V)
        gy0, gw0 = binding.invconv_backward(dev(gu), x0, wd)
        torch.cuda.synchronize()
        assert torch.equal(x, x0) and torch.equal(u, x) and torch.equal(gy, gy0) and torch.equal(gw, gw0)


def test_empty_batch_and_bad_arguments():
    import torch
    from paper_2410_14634_b200 import binding
    L = binding.lib()
    C, H, W, k = 2, 4, 4, 3
    w = dev(workloads.make_custom(9, 1, C, H, W, k)[0])
    s, b, V = dev(np.ones(C)), dev(np.zeros(C)), dev(np.eye(C))
    y = torch.empty(0, C, H, W, device="cuda")
    x, u, ld = binding.invconv_flow_step_forward(y, w, s, b, V)
    gy, gw, gs, gb, gV = binding.invconv_flow_step_backward(y, x, w, s, b, V)
    torch.cuda.synchronize()
    assert float(gw.abs().max()) == 0.0 and float(gV.abs().max()) == 0.0 and float(gs.abs().max()) == 0.0
    t = torch.zeros(4096, device="cuda")
    p = t.data_ptr()
    assert L.invconv_flow_step_forward(p, p, None, p, p, p + 4096, p + 8192, None, 1, 1, 4, 4, 3, None) == binding.BAD_ARG
    assert L.invconv_flow_step_forward(p, p, p, p, p, p, p + 8192, None, 1, 1, 4, 4, 3, None) == binding.BAD_ARG      # x aliases y
    assert L.invconv_flow_step_backward(p, p, p, p, p, p, p + 4096, None, p, p, p, 1, 1, 4, 4, 3, None) == binding.BAD_ARG
