"""Thin ctypes binding of libinvconv_b200.so: argument marshalling only.

Function names mirror the C ABI in `include/invconv.h`.  torch supplies device
memory and streams; every step of the computation runs inside the CUDA library.
There is no CPU or eager fallback: if the shared library is missing or a call
returns a non-zero status, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libinvconv_b200.so")

OK, BAD_ARG, UNSUPPORTED, CUDA_ERROR, TIMEOUT, WORKSPACE_TOO_SMALL, BOUNDS = range(7)
PATH_AUTO, PATH_GENERIC, PATH_WARP, PATH_TEAM, PATH_TENSOR = range(5)
WS_CONTROL_BYTES = 256

_lib = None


class InvConvError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        msg = lib().invconv_status_string(status).decode() if _lib is not None else str(status)
        super().__init__(f"{what}: status {status} ({msg})")


def lib() -> ctypes.CDLL:
    """Load the CUDA library (built by `paper_2410_14634_b200.build`)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2410_14634_b200.build` "
                "(there is no fallback path)")
        L = ctypes.CDLL(LIB_PATH)
        vp, fp, ci, sz = ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int, ctypes.c_size_t
        L.invconv_forward.argtypes = [fp, fp, fp, ci, ci, ci, ci, ci, vp]
        L.invconv_backward.argtypes = [fp, fp, fp, fp, fp, ci, ci, ci, ci, ci, vp]
        L.masked_conv_forward.argtypes = [fp, fp, fp, ci, ci, ci, ci, ci, vp]
        L.invconv_logdet.argtypes = [fp, fp, ci, ci, ci, ci, vp]
        L.invconv_forward_logdet.argtypes = [fp, fp, fp, fp, ci, ci, ci, ci, ci, vp]
        L.invconv_backward_logdet.argtypes = [fp, fp, fp, fp, fp, fp, ci, ci, ci, ci, ci, vp]
        L.invconv_flow_step_forward.argtypes = [fp] * 8 + [ci] * 5 + [vp]
        L.invconv_flow_step_forward.restype = ci
        L.invconv_flow_step_backward.argtypes = [fp] * 11 + [ci] * 5 + [vp]
        L.invconv_flow_step_backward.restype = ci
        L.invconv_forward_bf16.argtypes = [vp, fp, vp, ci, ci, ci, ci, ci, vp]
        L.invconv_forward_bf16.restype = ci
        L.invconv_backward_bf16.argtypes = [vp, vp, fp, vp, fp, ci, ci, ci, ci, ci, vp]
        L.invconv_backward_bf16.restype = ci
        L.invconv_bf16_in_kernel.argtypes = [ci] * 7
        L.invconv_bf16_in_kernel.restype = ci
        L.invconv_bf16_workspace_bytes.argtypes = [ci] * 5
        L.invconv_bf16_workspace_bytes.restype = sz
        L.invconv_forward_bf16_ws.argtypes = [vp, fp, vp, ci, ci, ci, ci, ci, vp, sz, vp]
        L.invconv_forward_bf16_ws.restype = ci
        L.invconv_backward_bf16_ws.argtypes = [vp, vp, fp, vp, fp, ci, ci, ci, ci, ci, vp, sz, vp]
        L.invconv_backward_bf16_ws.restype = ci
        L.invconv_workspace_bytes.argtypes = [ci] * 5
        L.invconv_workspace_bytes.restype = sz
        L.invconv_forward_ws.argtypes = [fp, fp, fp, ci, ci, ci, ci, ci, vp, sz, vp]
        L.invconv_backward_ws.argtypes = [fp, fp, fp, fp, fp, ci, ci, ci, ci, ci, vp, sz, vp]
        L.invconv_backward_noalloc.argtypes = [fp, fp, fp, fp, fp, ci, ci, ci, ci, ci, vp]
        L.invconv_backward_noalloc.restype = ci
        L.invconv_step_scratch_bytes.argtypes = [ci] * 5
        L.invconv_step_scratch_bytes.restype = sz
        L.invconv_step_host.argtypes = [vp] * 7 + [ci] * 5 + [vp, sz, vp]
        L.invconv_set_path.argtypes = [ci]
        L.invconv_set_option.argtypes = [ci, ci]
        L.invconv_set_option.restype = ci
        L.invconv_selftest_wait_timeout.argtypes = [ctypes.c_uint, vp]
        L.invconv_debug_bounds_info.argtypes = [ctypes.POINTER(ci)]
        L.invconv_debug_bounds_info.restype = ci
        L.invconv_selftest_bounds.argtypes = [vp]
        L.invconv_selftest_bounds.restype = ci
        L.invconv_selftest_wait_timeout.restype = ci
        L.invconv_path_for.argtypes = [ci] * 5
        L.invconv_cluster_size_for.argtypes = [ci] * 5
        L.invconv_cluster_size_for.restype = ci
        L.invconv_get_status.argtypes = [vp, ctypes.POINTER(ci)]
        L.invconv_probe_step_latency.argtypes = [ci, ci, vp, vp]
        L.invconv_status_string.argtypes = [ci]
        L.invconv_status_string.restype = ctypes.c_char_p
        L.invconv_version.argtypes = []
        L.invconv_kernel_launch_count.argtypes = []
        L.invconv_kernel_launch_count.restype = ctypes.c_ulonglong
        for name in ("invconv_forward", "invconv_backward", "masked_conv_forward", "invconv_logdet",
                     "invconv_forward_logdet", "invconv_backward_logdet",
                     "invconv_forward_ws", "invconv_backward_ws", "invconv_step_host", "invconv_set_path",
                     "invconv_path_for", "invconv_get_status", "invconv_probe_step_latency", "invconv_version"):
            getattr(L, name).restype = ci
        _lib = L
    return _lib


def _check(status: int, what: str) -> None:
    if status != OK:
        raise InvConvError(status, what)


def _stream_ptr(stream: Optional[torch.cuda.Stream], device) -> int:
    s = stream if stream is not None else torch.cuda.current_stream(device)
    return s.cuda_stream


def _act(t: torch.Tensor, name: str) -> torch.Tensor:
    if not (t.is_cuda and t.dtype == torch.float32 and t.dim() == 4 and t.is_contiguous()):
        raise ValueError(f"{name} must be a contiguous fp32 CUDA tensor [B,C,H,W]")
    return t


def _kern(w: torch.Tensor, C: int) -> int:
    if not (w.is_cuda and w.dtype == torch.float32 and w.dim() == 4 and w.is_contiguous()):
        raise ValueError("w must be a contiguous fp32 CUDA tensor [C,C,k,k]")
    if w.shape[0] != C or w.shape[1] != C or w.shape[2] != w.shape[3]:
        raise ValueError(f"w shape {tuple(w.shape)} does not match C={C}")
    return int(w.shape[2])


_workspaces: dict = {}


def workspace(B: int, C: int, H: int, W: int, k: int, device, stream_ptr: int, bf16: bool = False) -> Optional[torch.Tensor]:
    """A zero-initialised scratch tensor for this shape, cached per (device, stream); `bf16`: sized for the
    bfloat16-storage calls."""
    size_of = lib().invconv_bf16_workspace_bytes if bf16 else lib().invconv_workspace_bytes
    need = int(size_of(B, C, H, W, k))
    if need == 0:
        return None
    key = (torch.device(device).index, stream_ptr)
    ws = _workspaces.get(key)
    if ws is None or ws.numel() < need:
        ws = torch.zeros(need, dtype=torch.uint8, device=device)
        _workspaces[key] = ws
    return ws


def invconv_forward(y: torch.Tensor, w: torch.Tensor, out: Optional[torch.Tensor] = None,
                    stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
    """x = f^{-1}(y).  y [B,C,H,W], w [C,C,k,k]  ->  x [B,C,H,W]."""
    _act(y, "y")
    B, C, H, W = y.shape
    k = _kern(w, C)
    x = torch.empty_like(y) if out is None else _act(out, "out")
    with torch.cuda.device(y.device):
        sp = _stream_ptr(stream, y.device)
        ws = workspace(B, C, H, W, k, y.device, sp)
        _check(lib().invconv_forward_ws(y.data_ptr(), w.data_ptr(), x.data_ptr(), B, C, H, W, k,
                                        ws.data_ptr() if ws is not None else None,
                                        ws.numel() if ws is not None else 0, sp), "invconv_forward")
    return x


def invconv_backward(grad_x: torch.Tensor, x: torch.Tensor, w: torch.Tensor, need_grad_w: bool = True,
                     out_grad_y: Optional[torch.Tensor] = None, out_grad_w: Optional[torch.Tensor] = None,
                     stream: Optional[torch.cuda.Stream] = None):
    """(grad_y, grad_w) through x = f^{-1}(y), given grad_x and the saved x."""
    _act(grad_x, "grad_x")
    _act(x, "x")
    if grad_x.shape != x.shape:
        raise ValueError("grad_x and x must have the same shape")
    B, C, H, W = x.shape
    k = _kern(w, C)
    gy = torch.empty_like(grad_x) if out_grad_y is None else _act(out_grad_y, "out_grad_y")
    gw = None
    if need_grad_w:
        gw = torch.empty_like(w) if out_grad_w is None else out_grad_w
    with torch.cuda.device(x.device):
        sp = _stream_ptr(stream, x.device)
        ws = workspace(B, C, H, W, k, x.device, sp)
        _check(lib().invconv_backward_ws(grad_x.data_ptr(), x.data_ptr(), w.data_ptr(), gy.data_ptr(),
                                         gw.data_ptr() if gw is not None else None, B, C, H, W, k,
                                         ws.data_ptr() if ws is not None else None,
                                         ws.numel() if ws is not None else 0, sp), "invconv_backward")
    return gy, gw


NOALLOC_SCRATCH_BYTES = 1 << 20


def invconv_backward_noalloc(grad_x: torch.Tensor, x: torch.Tensor, w: torch.Tensor,
                             out_grad_y: torch.Tensor, out_grad_w: torch.Tensor,
                             stream: Optional[torch.cuda.Stream] = None) -> None:
    """`invconv_backward` for hosts that may no longer allocate device memory (a server with a frozen
    memory plan, a callback inside another framework): the caller passes every buffer, outputs included, and
    the library's scratch is a fixed array inside the library image (`NOALLOC_SCRATCH_BYTES`, shared by all
    calls on a device -- do not let two calls overlap on the GPU).  Raises `InvConvError` with status
    UNSUPPORTED or WORKSPACE_TOO_SMALL for shapes it does not serve; see `include/invconv.h`."""
    _act(grad_x, "grad_x"); _act(x, "x"); _act(out_grad_y, "out_grad_y")
    B, C, H, W = x.shape
    k = _kern(w, C)
    with torch.cuda.device(x.device):
        _check(lib().invconv_backward_noalloc(grad_x.data_ptr(), x.data_ptr(), w.data_ptr(), out_grad_y.data_ptr(),
                                              out_grad_w.data_ptr(), B, C, H, W, k, _stream_ptr(stream, x.device)),
               "invconv_backward_noalloc")


def masked_conv_forward(x: torch.Tensor, w: torch.Tensor, out: Optional[torch.Tensor] = None,
                        stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
    """y = f(x), the sampling direction."""
    _act(x, "x")
    B, C, H, W = x.shape
    k = _kern(w, C)
    y = torch.empty_like(x) if out is None else _act(out, "out")
    with torch.cuda.device(x.device):
        _check(lib().masked_conv_forward(x.data_ptr(), w.data_ptr(), y.data_ptr(), B, C, H, W, k,
                                         _stream_ptr(stream, x.device)), "masked_conv_forward")
    return y


def invconv_logdet(w: torch.Tensor, H: int, W: int, out: Optional[torch.Tensor] = None,
                   stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
    """H*W*sum_c log|w[c,c,k-1,k-1]| as a one-element fp32 CUDA tensor."""
    k = _kern(w, int(w.shape[0]))
    ld = torch.empty(1, dtype=torch.float32, device=w.device) if out is None else out
    with torch.cuda.device(w.device):
        _check(lib().invconv_logdet(w.data_ptr(), ld.data_ptr(), int(w.shape[0]), H, W, k,
                                    _stream_ptr(stream, w.device)), "invconv_logdet")
    return ld


def invconv_forward_logdet(y: torch.Tensor, w: torch.Tensor, stream: Optional[torch.cuda.Stream] = None):
    """(x, logdet): x = f^{-1}(y) and the log-det of f in one call."""
    _act(y, "y")
    B, C, H, W = y.shape
    k = _kern(w, C)
    x = torch.empty_like(y)
    ld = torch.empty(1, dtype=torch.float32, device=y.device)
    with torch.cuda.device(y.device):
        _check(lib().invconv_forward_logdet(y.data_ptr(), w.data_ptr(), x.data_ptr(), ld.data_ptr(), B, C, H, W, k,
                                            _stream_ptr(stream, y.device)), "invconv_forward_logdet")
    return x, ld


def invconv_backward_logdet(grad_x: torch.Tensor, x: torch.Tensor, w: torch.Tensor, grad_logdet: torch.Tensor,
                            stream: Optional[torch.cuda.Stream] = None):
    """(grad_y, grad_w) with grad_logdet * d logdet / d w added to grad_w; grad_logdet is a one-element fp32
    CUDA tensor (the upstream gradient with respect to the log-det)."""
    _act(grad_x, "grad_x")
    _act(x, "x")
    if grad_x.shape != x.shape:
        raise ValueError("grad_x and x must have the same shape")
    if grad_logdet.dtype != torch.float32 or grad_logdet.numel() != 1 or not grad_logdet.is_cuda:
        raise ValueError("grad_logdet must be a one-element fp32 CUDA tensor")
    B, C, H, W = x.shape
    k = _kern(w, C)
    gy, gw = torch.empty_like(grad_x), torch.empty_like(w)
    with torch.cuda.device(x.device):
        _check(lib().invconv_backward_logdet(grad_x.data_ptr(), x.data_ptr(), w.data_ptr(), grad_logdet.data_ptr(),
                                             gy.data_ptr(), gw.data_ptr(), B, C, H, W, k,
                                             _stream_ptr(stream, x.device)), "invconv_backward_logdet")
    return gy, gw


def invconv_flow_step_forward(y: torch.Tensor, w: torch.Tensor, s: torch.Tensor, b: torch.Tensor, V: torch.Tensor,
                              want_logdet: bool = True, stream: Optional[torch.cuda.Stream] = None):
    """(x, u, logdet) of one flow step: x = f^{-1}(y), u = V (s * x + b); logdet is a one-element tensor or None."""
    _act(y, "y")
    B, C, H, W = y.shape
    k = _kern(w, C)
    x, u = torch.empty_like(y), torch.empty_like(y)
    ld = torch.empty(1, dtype=torch.float32, device=y.device) if want_logdet else None
    with torch.cuda.device(y.device):
        _check(lib().invconv_flow_step_forward(y.data_ptr(), w.data_ptr(), s.data_ptr(), b.data_ptr(), V.data_ptr(),
                                               x.data_ptr(), u.data_ptr(), ld.data_ptr() if ld is not None else None,
                                               B, C, H, W, k, _stream_ptr(stream, y.device)), "invconv_flow_step_forward")
    return x, u, ld


def invconv_flow_step_backward(grad_u: torch.Tensor, x: torch.Tensor, w: torch.Tensor, s: torch.Tensor, b: torch.Tensor,
                               V: torch.Tensor, stream: Optional[torch.cuda.Stream] = None):
    """(grad_y, grad_w, grad_s, grad_b, grad_V) through one flow step, given grad_u and the saved x."""
    _act(grad_u, "grad_u")
    _act(x, "x")
    B, C, H, W = x.shape
    k = _kern(w, C)
    gy, gw = torch.empty_like(x), torch.empty_like(w)
    gs, gb, gV = torch.empty_like(s), torch.empty_like(b), torch.empty_like(V)
    with torch.cuda.device(x.device):
        _check(lib().invconv_flow_step_backward(grad_u.data_ptr(), x.data_ptr(), w.data_ptr(), s.data_ptr(), b.data_ptr(),
                                                V.data_ptr(), gy.data_ptr(), gw.data_ptr(), gs.data_ptr(), gb.data_ptr(),
                                                gV.data_ptr(), B, C, H, W, k, _stream_ptr(stream, x.device)),
               "invconv_flow_step_backward")
    return gy, gw, gs, gb, gV


def _act16(t: torch.Tensor, name: str) -> torch.Tensor:
    if not (t.is_cuda and t.dtype == torch.bfloat16 and t.dim() == 4 and t.is_contiguous()):
        raise ValueError(f"{name} must be a contiguous bfloat16 CUDA tensor [B,C,H,W]")
    return t


def invconv_forward_bf16(y: torch.Tensor, w: torch.Tensor, out: Optional[torch.Tensor] = None,
                         stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
    """x = f^{-1}(y) with bfloat16 activations in memory (fp32 weights, fp32 arithmetic)."""
    _act16(y, "y")
    B, C, H, W = y.shape
    k = _kern(w, C)
    x = torch.empty_like(y) if out is None else _act16(out, "out")
    with torch.cuda.device(y.device):
        sp = _stream_ptr(stream, y.device)
        if (y.data_ptr() | x.data_ptr()) & 15 or B == 0:
            # buffers off a 16-byte boundary: the library sizes its own scratch for the route it has to take
            _check(lib().invconv_forward_bf16(y.data_ptr(), w.data_ptr(), x.data_ptr(), B, C, H, W, k, sp), "invconv_forward_bf16")
        else:
            ws = workspace(B, C, H, W, k, y.device, sp, bf16=True)
            _check(lib().invconv_forward_bf16_ws(y.data_ptr(), w.data_ptr(), x.data_ptr(), B, C, H, W, k,
                                                 ws.data_ptr(), ws.numel(), sp), "invconv_forward_bf16")
    return x


def invconv_backward_bf16(grad_x: torch.Tensor, x: torch.Tensor, w: torch.Tensor, need_grad_w: bool = True,
                          out_grad_y: Optional[torch.Tensor] = None, out_grad_w: Optional[torch.Tensor] = None,
                          stream: Optional[torch.cuda.Stream] = None):
    """(grad_y, grad_w) with bfloat16 activations in memory; grad_w is fp32 (None if not asked for)."""
    _act16(grad_x, "grad_x")
    _act16(x, "x")
    B, C, H, W = x.shape
    k = _kern(w, C)
    gy = torch.empty_like(x) if out_grad_y is None else _act16(out_grad_y, "out_grad_y")
    gw = (out_grad_w if out_grad_w is not None else torch.empty_like(w)) if need_grad_w else None
    with torch.cuda.device(x.device):
        sp = _stream_ptr(stream, x.device)
        gwp = gw.data_ptr() if gw is not None else None
        if (grad_x.data_ptr() | x.data_ptr() | gy.data_ptr()) & 15 or B == 0:
            _check(lib().invconv_backward_bf16(grad_x.data_ptr(), x.data_ptr(), w.data_ptr(), gy.data_ptr(), gwp,
                                               B, C, H, W, k, sp), "invconv_backward_bf16")
        else:
            ws = workspace(B, C, H, W, k, x.device, sp, bf16=True)
            _check(lib().invconv_backward_bf16_ws(grad_x.data_ptr(), x.data_ptr(), w.data_ptr(), gy.data_ptr(), gwp,
                                                  B, C, H, W, k, ws.data_ptr(), ws.numel(), sp), "invconv_backward_bf16")
    return gy, gw


def invconv_bf16_in_kernel(B: int, C: int, H: int, W: int, k: int, backward: bool = False, with_grad_w: bool = True) -> bool:
    return bool(lib().invconv_bf16_in_kernel(B, C, H, W, k, int(backward), int(with_grad_w)))


class HostStep:
    """One layer step (forward, backward, log-det) from pinned HOST buffers
    through `invconv_step_host`: the copies to and from the device are part of
    the call.  Holds the pinned buffers and the device scratch for one shape."""

    def __init__(self, B: int, C: int, H: int, W: int, k: int, device="cuda:0"):
        self.shape = (B, C, H, W, k)
        self.device = torch.device(device)
        pin = dict(dtype=torch.float32, pin_memory=True)
        self.y = torch.empty(B, C, H, W, **pin)
        self.grad_x = torch.empty(B, C, H, W, **pin)
        self.w = torch.empty(C, C, k, k, **pin)
        self.x = torch.empty(B, C, H, W, **pin)
        self.grad_y = torch.empty(B, C, H, W, **pin)
        self.grad_w = torch.empty(C, C, k, k, **pin)
        self.logdet = torch.empty(1, **pin)
        n = int(lib().invconv_step_scratch_bytes(B, C, H, W, k))
        self.scratch = torch.zeros(n, dtype=torch.uint8, device=self.device)
        self.h2d_bytes = 4 * (self.y.numel() + self.grad_x.numel() + self.w.numel())
        self.d2h_bytes = 4 * (self.x.numel() + self.grad_y.numel() + self.grad_w.numel() + 1)

    def run(self, stream: Optional[torch.cuda.Stream] = None) -> None:
        """Enqueue one step; synchronise the stream before reading the outputs."""
        B, C, H, W, k = self.shape
        with torch.cuda.device(self.device):
            _check(lib().invconv_step_host(self.y.data_ptr(), self.w.data_ptr(), self.grad_x.data_ptr(),
                                           self.x.data_ptr(), self.grad_y.data_ptr(), self.grad_w.data_ptr(),
                                           self.logdet.data_ptr(), B, C, H, W, k, self.scratch.data_ptr(),
                                           self.scratch.numel(), _stream_ptr(stream, self.device)),
                   "invconv_step_host")


# invconv_option values (development and test controls, see include/invconv.h)
(OPT_WARP_RING, OPT_WARP_CHANNEL_SPLIT, OPT_GRADW_SEPARATE, OPT_GRADW_TENSOR_PIPE, OPT_TEAM_VARIANT,
 OPT_TEAM_CLUSTER, OPT_DEPENDENT_LAUNCH) = range(7)


def invconv_set_option(option: int, value: int) -> int:
    """Set a development/test control; returns the previous value."""
    prev = int(lib().invconv_set_option(option, value))
    if prev == -1 and not (0 <= option < 7):
        raise ValueError("unknown option")
    return prev


def invconv_selftest_wait_timeout(limit_cycles: int = 20000, stream: Optional[torch.cuda.Stream] = None,
                                  device="cuda:0") -> None:
    """Launch the kernel whose bounded wait runs out on purpose (see include/invconv.h)."""
    with torch.cuda.device(device):
        _check(lib().invconv_selftest_wait_timeout(limit_cycles, _stream_ptr(stream, device)),
               "invconv_selftest_wait_timeout")


def invconv_debug_bounds_info():
    """(site, index, limit, count) of the debug-bounds build's record (cleared by the call); None in the normal build."""
    arr = (ctypes.c_int * 4)()
    rc = int(lib().invconv_debug_bounds_info(arr))
    if rc == UNSUPPORTED:
        return None
    _check(rc, "invconv_debug_bounds_info")
    return tuple(int(v) for v in arr)


def invconv_set_path(path: int) -> int:
    return int(lib().invconv_set_path(path))


def invconv_path_for(B: int, C: int, H: int, W: int, k: int) -> int:
    return int(lib().invconv_path_for(B, C, H, W, k))


def invconv_cluster_size_for(B: int, C: int, H: int, W: int, k: int) -> int:
    return int(lib().invconv_cluster_size_for(B, C, H, W, k))


def invconv_get_status(stream: Optional[torch.cuda.Stream] = None, device="cuda:0") -> int:
    out = ctypes.c_int(0)
    with torch.cuda.device(device):
        _check(lib().invconv_get_status(_stream_ptr(stream, device), ctypes.byref(out)), "invconv_get_status")
    return out.value


def invconv_probe_step_latency(mechanism: int, steps: int = 4096, device="cuda:0") -> float:
    """SM clock cycles per dependent wavefront step for a mechanism (0 shuffle, 1 shared memory + block barrier,
    2 cluster shared memory + cluster barrier)."""
    buf = torch.zeros(2, dtype=torch.int64, device=device)
    with torch.cuda.device(device):
        _check(lib().invconv_probe_step_latency(mechanism, steps, buf.data_ptr(), _stream_ptr(None, device)),
               "invconv_probe_step_latency")
        torch.cuda.synchronize()
    return float(buf[0].item()) / steps


def invconv_kernel_launch_count() -> int:
    return int(lib().invconv_kernel_launch_count())


def invconv_version() -> int:
    return int(lib().invconv_version())
