"""Several host threads, each on its own stream, call the library at once on shapes of every kernel family: results
must equal those of the same calls made alone, bit for bit (per-stream workspaces in the binding, the library's
scratch pool, cached per-device state and the control words in the workspaces are all shared between the threads)."""
import threading
import time

import numpy as np
import pytest

from paper_2410_14634_b200 import workloads

pytestmark = pytest.mark.gpu

SHAPES = [(8, 1, 28, 28, 3), (6, 3, 32, 32, 3), (9, 48, 16, 16, 3), (4, 12, 16, 16, 3), (3, 96, 8, 8, 3), (2, 3, 64, 64, 5),
          (16, 16, 8, 8, 5), (2, 1, 200, 180, 5)]


def test_concurrent_streams_reproduce_the_serial_results():
    import torch
    from paper_2410_14634_b200 import binding
    data = []
    for i, sh in enumerate(SHAPES):
        C = sh[1]
        w, y, gx = workloads.make_custom(i, *sh, sigma=0.05 / np.sqrt(C))
        wd, yd, gxd = (torch.from_numpy(a).cuda() for a in (w, y, gx))
        ident = (torch.ones(C, device="cuda"), torch.zeros(C, device="cuda"), torch.eye(C, device="cuda"))
        x = binding.invconv_forward(yd, wd)
        gy, gw = binding.invconv_backward(gxd, x, wd)
        f = binding.masked_conv_forward(x, wd)
        _, u, _ = binding.invconv_flow_step_forward(yd, wd, *ident)
        torch.cuda.synchronize()
        data.append((wd, yd, gxd, ident, x, gy, gw, f, u))
    mismatches, counts = [], []
    stop = time.time() + 4.0

    def worker(tid):
        rng = np.random.default_rng(tid)
        stream = torch.cuda.Stream()
        done = 0
        with torch.cuda.stream(stream):
            while time.time() < stop:
                i = int(rng.integers(len(SHAPES)))
                wd, yd, gxd, ident, x0, gy0, gw0, f0, u0 = data[i]
                x = binding.invconv_forward(yd, wd)
                gy, gw = binding.invconv_backward(gxd, x, wd)
                f = binding.masked_conv_forward(x, wd)
                _, u, _ = binding.invconv_flow_step_forward(yd, wd, *ident)
                stream.synchronize()
                if not (torch.equal(x, x0) and torch.equal(gy, gy0) and torch.equal(gw, gw0) and torch.equal(f, f0) and torch.equal(u, u0)):
                    mismatches.append((tid, SHAPES[i]))
                done += 1
        counts.append(done)

    threads = [threading.Thread(target=worker, args=(t,)) for t in range(4)]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    torch.cuda.synchronize()
    assert binding.invconv_get_status() == 0
    assert not mismatches, mismatches[:5]
    assert len(counts) == 4 and min(counts) > 10
