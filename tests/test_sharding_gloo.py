"""The multi-process path on CPU (gloo, world size 2): batch sharding, the grad_w all-reduce and the
max-over-ranks timing reduction used by bench.py under torchrun."""
import os
import socket

import numpy as np
import pytest

torch = pytest.importorskip("torch")
import torch.multiprocessing as mp  # noqa: E402

from paper_2410_14634_b200 import sharding, workloads  # noqa: E402


def test_shard_batch_partitions_the_batch():
    for B in (0, 1, 5, 64, 257):
        for world in (1, 2, 3, 8):
            spans = [sharding.shard_batch(B, world, r) for r in range(world)]
            assert spans[0][0] == 0 and sum(c for _, c in spans) == B
            for (s0, c0), (s1, _) in zip(spans, spans[1:]):
                assert s0 + c0 == s1
            assert max(c for _, c in spans) - min(c for _, c in spans) <= 1


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    import torch.distributed as dist
    from oracle import api
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        s, w, y, gx = workloads.make("pr1")
        start, count = sharding.shard_batch(s.B, world, rank)
        ys, gxs = y[start:start + count], gx[start:start + count]
        x = api.invconv_forward(ys, w)
        gy, gw = api.invconv_backward(gxs, x, w)
        gw_t = torch.from_numpy(gw.copy())
        sharding.allreduce_grad_w(gw_t)
        slow = sharding.max_over_ranks(1.0 + rank)
        if rank == 0:
            out.put((gw_t.numpy(), slow))
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_ranks_reproduce_the_full_batch_grad_w():
    from oracle import api
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    gw_sum, slow = out.get(timeout=120)
    for p in procs:
        p.join(timeout=120)
        assert p.exitcode == 0
    s, w, y, gx = workloads.make("pr1")
    x = api.invconv_forward(y, w)
    _, gw_full = api.invconv_backward(gx, x, w)
    assert np.max(np.abs(gw_sum - gw_full)) <= 1e-12 * max(1.0, np.max(np.abs(gw_full)))
    assert slow == 2.0
