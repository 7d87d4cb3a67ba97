"""Host logic of the N > 1 path on CPU: two gloo ranks shard the (batch, head) units with no
data-path collective and reduce only the timing (max over ranks), as bench.py does with NCCL."""
import os
import socket
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2609_04105_b200 import inputs as I

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_shard_units_partitions_exactly():
    for n in (1, 7, 64, 128):
        for world in (1, 2, 3, 8):
            spans = [I.shard_units(n, world, r) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == n
            assert all(a[1] == b[0] for a, b in zip(spans[:-1], spans[1:]))
            sizes = [e - b for b, e in spans]
            assert max(sizes) - min(sizes) <= 1


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from oracle import attention as A
    from oracle import quantize as Qz
    w = I.shrink(I.WORKLOADS["cfg1"], H=4, N=128)
    q, k, v = I.make_qkv(w)
    qd, kd, vd = Qz.quantize_qk(q, "mx"), Qz.quantize_qk(k, "mx"), Qz.quantize_v(v)
    units = [(b, h) for b in range(w.B) for h in range(w.H)]
    lo, hi = I.shard_units(len(units), world, rank)
    O, _ = A.direct_p_forward(qd, kd, vd, heads=units[lo:hi])          # this rank's independent units
    t = torch.tensor([float(rank + 1)], dtype=torch.float64)            # stand-in for elapsed ms
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    gathered = [None] * world
    dist.all_gather_object(gathered, (lo, hi, O))
    if rank == 0:
        full = np.concatenate([g[2] for g in sorted(gathered, key=lambda g: g[0])])
        ref, _ = A.direct_p_forward(qd, kd, vd)
        out.put((float(t[0]), bool(np.array_equal(full, ref)), [g[:2] for g in gathered]))
    dist.destroy_process_group()


def test_two_ranks_cover_all_units_and_time_is_max_over_ranks():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = out.get(timeout=240)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    tmax, same, spans = res
    assert tmax == 2.0                      # max over ranks, not rank 0's own value
    assert same                             # sharded units reassemble to the unsharded result
    assert sorted(spans) == [(0, 2), (2, 4)]
