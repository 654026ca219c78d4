"""The N > 1 path on CPU: gloo ranks partition the (batch, head) units through the same helper the
GPU path uses (monarch_attn_fwd_sharded), each computes its own shard (a CPU stand-in takes the
place of the library call: the partition and the gather are what is exercised here), and the pieces
reassemble to the single-process result with no data-path collective."""
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


def _stand_in(Qs, Ks, Vs, b, T):
    """What the library call computes, on the host: [1, units, N, d] -> [1, units, N, d]."""
    return torch.from_numpy(mo.monarch_attention(Qs.numpy(), Ks.numpy(), Vs.numpy(), b, T))


def _worker(rank, world, port, q, shape):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank),
                      LOCAL_RANK=str(rank), WORLD_SIZE=str(world))
    r, _, w = D.init("gloo")
    assert (r, w) == (rank, world)
    batch, heads, N, d, b, T = shape
    Q, K, V = (torch.from_numpy(x).double() for x in wl.make_qkv(batch, heads, N, d, "f32", 2, 1.0, seed=9))
    mine, (lo, hi) = D.monarch_attn_fwd_sharded(Q, K, V, b, T, gather=False, fwd=_stand_in)
    assert mine.shape == (hi - lo, N, d) and (lo, hi) == D.my_units(batch * heads)
    D.barrier()
    step_time = D.max_over_ranks(1.0 + rank)            # max over ranks, as the benchmark does
    full = D.monarch_attn_fwd_sharded(Q, K, V, b, T, gather=True, fwd=_stand_in)
    if rank == 0:
        q.put((lo, hi, step_time, full.numpy()))
    D.barrier()
    torch.distributed.destroy_process_group()


def _run(world, shape):
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q, shape)) for r in range(world)]
    for p in procs:
        p.start()
    out = q.get(timeout=120)
    for p in procs:
        p.join(timeout=120)
        assert p.exitcode == 0
    return out


def test_two_gloo_ranks_partition_heads_and_reassemble():
    shape = (3, 3, 24, 4, 6, 2)
    lo, hi, step_time, full = _run(2, shape)
    assert (lo, hi) == (0, 5) and step_time == 2.0
    Q, K, V = wl.make_qkv(3, 3, 24, 4, "f32", 2, 1.0, seed=9)
    ref = mo.monarch_attention(Q.astype(np.float64), K.astype(np.float64), V.astype(np.float64), 6, 2)
    assert np.array_equal(full, ref)


def test_more_ranks_than_units_leaves_some_ranks_idle():
    shape = (1, 2, 12, 4, 4, 1)
    lo, hi, step_time, full = _run(3, shape)
    assert (lo, hi) == (0, 1) and step_time == 3.0
    Q, K, V = wl.make_qkv(1, 2, 12, 4, "f32", 2, 1.0, seed=9)
    ref = mo.monarch_attention(Q.astype(np.float64), K.astype(np.float64), V.astype(np.float64), 4, 1)
    assert np.array_equal(full, ref)


def test_without_a_process_group_it_is_the_single_process_call():
    Q, K, V = (torch.from_numpy(x).double() for x in wl.make_qkv(2, 2, 12, 4, "f32", 2, 1.0, seed=3))
    full = D.monarch_attn_fwd_sharded(Q, K, V, 4, 2, fwd=_stand_in)
    assert np.array_equal(full.numpy(), mo.monarch_attention(Q.numpy(), K.numpy(), V.numpy(), 4, 2))
