"""The N > 1 path on CPU: two gloo ranks partition the (batch, head) units, each computes its own
shard (with the oracle standing in for the GPU call), and the pieces reassemble to the
single-process result with no data-path collective."""
import os
import socket

import numpy as np
import torch
import torch.multiprocessing as mp

from oracle import monarch_oracle as mo
from paper_2505_18698_b200 import distributed as D, workloads as wl


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank),
                      LOCAL_RANK=str(rank), WORLD_SIZE=str(world))
    r, _, w = D.init("gloo")
    assert (r, w) == (rank, world)
    batch, heads, N, d, b, T = 3, 3, 24, 4, 6, 2
    Q, K, V = wl.make_qkv(batch, heads, N, d, "f32", 2, 1.0, seed=9)
    total = batch * heads
    lo, hi = D.my_units(total)
    flat = lambda x: x.reshape(total, N, d)
    mine = mo.monarch_attention(flat(Q)[lo:hi], flat(K)[lo:hi], flat(V)[lo:hi], b, T)
    D.barrier()
    step_time = D.max_over_ranks(1.0 + rank)            # max over ranks, as the benchmark does
    full = D.gather_units(torch.from_numpy(mine), total).numpy()
    if rank == 0:
        q.put((lo, hi, step_time, full))
    D.barrier()
    torch.distributed.destroy_process_group()


def test_two_gloo_ranks_partition_heads_and_reassemble():
    world = 2
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    lo, hi, step_time, full = q.get(timeout=120)
    for p in procs:
        p.join(timeout=120)
        assert p.exitcode == 0
    assert (lo, hi) == (0, 5) and step_time == 2.0
    Q, K, V = wl.make_qkv(3, 3, 24, 4, "f32", 2, 1.0, seed=9)
    ref = mo.monarch_attention(Q, K, V, 6, 2).reshape(9, 24, 4)
    assert np.array_equal(full, ref)
