"""Parity of the bfloat16-storage calls with the float64 oracle, through the C ABI: shapes whose wavefront kernel
reads and writes bfloat16 itself (one warp per image, several warps, several images per CTA, the channel-split
walk, with and without grad_w riding along) and shapes composed around the fp32 path (images in global memory,
grad_w from the separate kernel, the team, tensor and generic families, sizes off the 8-value unit).

Both sides see the same bfloat16 inputs (exact in float64).  An output value may differ from the oracle's
rounded value only by the rounding itself plus the fp32 path's own error:
    |out - ref| <= spacing(ref) / 2 + 1e-4 * max|ref|          (spacing = distance of neighbouring bfloat16 values)
and where the reference is farther than that error from a rounding boundary the stored value must be exactly
the oracle's rounded value (checked as: at least 99 % of the values agree exactly)."""
import numpy as np
import pytest

from conftest import nmax_err
from paper_2410_14634_b200 import workloads

pytestmark = pytest.mark.gpu

# (shape, handled inside the wavefront kernel for forward / backward with grad_w)
IN_KERNEL = [(8, 1, 28, 28, 3), (6, 3, 32, 32, 3), (4, 3, 16, 16, 3), (3, 2, 40, 36, 3), (2, 3, 64, 64, 5),
             (5, 4, 8, 8, 2), (3, 1, 64, 64, 5), (256, 1, 28, 28, 3)]
COMPOSED = [(2, 1, 250, 256, 3), (4, 12, 16, 16, 3), (9, 48, 16, 16, 3), (3, 96, 8, 8, 3), (2, 3, 9, 11, 3),
            (1, 5, 6, 7, 3), (2, 3, 16, 16, 7)]


def to16(a):
    import torch
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(torch.bfloat16).cuda()


def as64(t):
    import torch
    return t.to(torch.float64).cpu().numpy()


def check_stored(out, ref, what):
    from oracle import storage
    scale = float(np.max(np.abs(ref)))
    bound = 0.5 * storage.bf16_spacing(ref) + 1e-4 * scale
    err = np.abs(out - ref)
    assert np.all(err <= bound), f"{what}: worst excess {float(np.max(err - bound)):.3e}"
    agree = float(np.mean(out == storage.round_to_bf16(ref)))
    assert agree >= 0.99, f"{what}: only {agree:.4f} of the values equal the oracle's rounded value"


@pytest.mark.parametrize("shape", IN_KERNEL + COMPOSED, ids=lambda s: "x".join(map(str, s)))
def test_bf16_storage_matches_oracle(shape):
    import torch
    from paper_2410_14634_b200 import binding
    from oracle import api as oracle
    Bn, C, H, W, k = shape
    w, y, gx = workloads.make_custom(900 + sum(shape), Bn, C, H, W, k, sigma=0.05 / np.sqrt(C))
    y16, gx16, wd = to16(y), to16(gx), torch.from_numpy(w).cuda()
    x_ref = oracle.invconv_forward(as64(y16), w)
    for _ in range(2):                      # twice: scratch and control words are left reusable
        x16 = binding.invconv_forward_bf16(y16, wd)
        gy16, gw = binding.invconv_backward_bf16(gx16, x16, wd)
        gy16_only, none = binding.invconv_backward_bf16(gx16, x16, wd, need_grad_w=False)
        torch.cuda.synchronize()
        assert binding.invconv_get_status() == 0 and none is None
        check_stored(as64(x16), x_ref, "x")
        # the backward call sees the stored x, as a training step does
        gy_ref, gw_ref = oracle.invconv_backward(as64(gx16), as64(x16), w)
        check_stored(as64(gy16), gy_ref, "grad_y")
        assert torch.equal(gy16, gy16_only)
        assert nmax_err(gw.cpu().numpy(), gw_ref) <= 1e-3
        mask = np.triu(np.ones((C, C), dtype=bool), 1)
        assert np.all(gw.cpu().numpy()[:, :, k - 1, k - 1][mask] == 0.0)


def test_which_shapes_run_inside_the_kernel():
    from paper_2410_14634_b200 import binding
    for s in IN_KERNEL:
        assert binding.invconv_bf16_in_kernel(*s, backward=False)
        assert binding.invconv_bf16_in_kernel(*s, backward=True, with_grad_w=False)
    # grad_w rides along only where its sums fit the wavefront's registers
    assert binding.invconv_bf16_in_kernel(6, 3, 32, 32, 3, backward=True, with_grad_w=True)
    assert not binding.invconv_bf16_in_kernel(2, 3, 64, 64, 5, backward=True, with_grad_w=True)
    for s in COMPOSED:
        assert not binding.invconv_bf16_in_kernel(*s, backward=False)


def test_bf16_storage_agrees_with_the_fp32_calls_on_the_same_values():
    """Same inputs (bfloat16 values held in fp32 buffers) through the fp32 calls, rounded by the library's own
    conversion: the stored results must be identical -- the variant changes the format in memory only."""
    import torch
    from paper_2410_14634_b200 import binding
    for shape in [(8, 1, 28, 28, 3), (6, 3, 32, 32, 3), (9, 48, 16, 16, 3)]:
        Bn, C, H, W, k = shape
        w, y, gx = workloads.make_custom(77 + sum(shape), Bn, C, H, W, k, sigma=0.05 / np.sqrt(C))
        y16, gx16, wd = to16(y), to16(gx), torch.from_numpy(w).cuda()
        x16 = binding.invconv_forward_bf16(y16, wd)
        x32 = binding.invconv_forward(y16.float(), wd)
        assert torch.equal(x16, x32.to(torch.bfloat16))
        gy16, gw16 = binding.invconv_backward_bf16(gx16, x16, wd)
        gy32, gw32 = binding.invconv_backward(gx16.float(), x16.float(), wd)
        assert torch.equal(gy16, gy32.to(torch.bfloat16))
        assert torch.equal(gw16, gw32)


def test_bf16_storage_with_buffers_off_a_16_byte_boundary():
    """Buffers 2 bytes off: the wavefront kernel's bulk copies cannot take them, the composed route serves them."""
    import torch
    from paper_2410_14634_b200 import binding
    from oracle import api as oracle
    for shape in [(6, 3, 32, 32, 3), (9, 48, 16, 16, 3)]:
        Bn, C, H, W, k = shape
        w, y, gx = workloads.make_custom(31 + sum(shape), Bn, C, H, W, k, sigma=0.05 / np.sqrt(C))
        wd = torch.from_numpy(w).cuda()

        def off(a=None):
            buf = torch.empty(y.size + 1, dtype=torch.bfloat16, device="cuda")
            v = buf[1:].view(y.shape)
            if a is not None:
                v.copy_(torch.from_numpy(a))
            return v

        y16, gx16, x16, gy16 = off(y), off(gx), off(), off()
        binding.invconv_forward_bf16(y16, wd, out=x16)
        _, gw = binding.invconv_backward_bf16(gx16, x16, wd, out_grad_y=gy16)
        torch.cuda.synchronize()
        assert binding.invconv_get_status() == 0
        check_stored(as64(x16), oracle.invconv_forward(as64(y16), w), "x")
        gy_ref, gw_ref = oracle.invconv_backward(as64(gx16), as64(x16), w)
        check_stored(as64(gy16), gy_ref, "grad_y")
        assert nmax_err(gw.cpu().numpy(), gw_ref) <= 1e-3


def test_bf16_workspace_forms_reject_a_short_workspace():
    import torch
    from paper_2410_14634_b200 import binding
    L = binding.lib()
    for shape in [(6, 3, 32, 32, 3), (4, 12, 16, 16, 3)]:
        Bn, C, H, W, k = shape
        need = L.invconv_bf16_workspace_bytes(*shape)
        assert need >= L.invconv_workspace_bytes(*shape) > 0
        ws = torch.zeros(need, dtype=torch.uint8, device="cuda")
        y = torch.zeros(Bn, C, H, W, device="cuda", dtype=torch.bfloat16)
        x = torch.empty_like(y)
        w = torch.eye(C, device="cuda").reshape(C, C, 1, 1).repeat(1, 1, k, k).contiguous()
        assert L.invconv_forward_bf16_ws(y.data_ptr(), w.data_ptr(), x.data_ptr(), *shape, ws.data_ptr(), need, None) == binding.OK
        assert L.invconv_forward_bf16_ws(y.data_ptr(), w.data_ptr(), x.data_ptr(), *shape, ws.data_ptr(), 128, None) == binding.WORKSPACE_TOO_SMALL
        assert L.invconv_backward_bf16_ws(y.data_ptr(), x.data_ptr(), w.data_ptr(), y.data_ptr(), None, *shape, ws.data_ptr(), need, None) == binding.BAD_ARG
        gy = torch.empty_like(y)
        assert L.invconv_backward_bf16_ws(y.data_ptr(), x.data_ptr(), w.data_ptr(), gy.data_ptr(), None, *shape, None, 0, None) == binding.WORKSPACE_TOO_SMALL
        torch.cuda.synchronize()


def test_bf16_storage_empty_batch_and_bad_arguments():
    import torch
    from paper_2410_14634_b200 import binding
    L = binding.lib()
    w = torch.ones(1, 1, 3, 3, device="cuda")
    gw = torch.full((1, 1, 3, 3), 7.0, device="cuda")
    assert L.invconv_forward_bf16(None, w.data_ptr(), None, 0, 1, 8, 8, 3, None) == binding.OK
    assert L.invconv_backward_bf16(None, None, w.data_ptr(), None, gw.data_ptr(), 0, 1, 8, 8, 3, None) == binding.OK
    torch.cuda.synchronize()
    assert float(gw.abs().sum()) == 0.0
    y = torch.zeros(1, 1, 8, 8, device="cuda", dtype=torch.bfloat16)
    assert L.invconv_forward_bf16(y.data_ptr(), w.data_ptr(), y.data_ptr(), 1, 1, 8, 8, 3, None) == binding.BAD_ARG
    assert L.invconv_forward_bf16(None, w.data_ptr(), y.data_ptr(), 1, 1, 8, 8, 3, None) == binding.BAD_ARG
    assert L.invconv_backward_bf16(y.data_ptr(), y.data_ptr(), w.data_ptr(), y.data_ptr(), None, 1, 1, 8, 8, 3, None) == binding.BAD_ARG
