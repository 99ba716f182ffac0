"""world_size-2 gloo test of the data-parallel plumbing on CPU: row shards need no exchange on the
forward path, and the backward's gain gradient is one all-reduce of D floats."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2603_13180_b200 import sharding
from paper_2603_13180_b200 import workloads as wl


def test_shard_rows_partition():
    for T in (0, 1, 127, 128, 129, 1000, 16384, 16385):
        for world in (1, 2, 3, 8):
            spans = [sharding.shard_rows(T, r, world) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == T
            for (b0, e0), (b1, e1) in zip(spans, spans[1:]):
                assert e0 == b1 and b0 <= e0
            assert all(b % 128 == 0 for b, _ in spans if b < T)
            sizes = [e - b for b, e in spans]
            assert max(sizes) - min(sizes) < 2 * 128   # one tile of imbalance plus the ragged last tile
    assert sharding.shard_rows(16384, 3, 8) == (6144, 8192)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, T, D, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        import oracle
        w = wl.Workload("t", T, D, seed=3, outlier_frac=0.004, has_gain=True, has_grad=True)
        inp = wl.make_inputs(w)                       # same seed on every rank -> same global tensors
        x, g, gain = wl.bits(inp["x"]), wl.bits(inp["grad"]), wl.bits(inp["gain"])
        b, e = sharding.shard_rows(T, rank, world)
        codes, scales, rms = oracle.mxnorm_ref(x[b:e], eps=1e-5)
        _, dg = oracle.mxnorm_bwd_ref(x[b:e], g[b:e], gain, rms, want_dx=False)
        dg_t = torch.from_numpy(dg.copy())
        sharding.allreduce_dgain(dg_t)                # the backward's only exchange
        slow = sharding.max_over_ranks(1.0 + rank)    # timing reduction: max over ranks
        gathered = [None] * world
        dist.all_gather_object(gathered, (b, e, codes, scales, rms))   # test-only gather to compare with the unsharded run
        if rank == 0:
            full_codes, full_scales, full_rms = oracle.mxnorm_ref(x, eps=1e-5)
            _, full_dg = oracle.mxnorm_bwd_ref(x, g, gain, full_rms, want_dx=False)
            cat = lambda i: np.concatenate([gathered[r][i] for r in range(world)])
            ok = (np.array_equal(cat(2), full_codes) and np.array_equal(cat(3), full_scales)
                  and np.array_equal(cat(4), full_rms)
                  and np.allclose(dg_t.numpy(), full_dg, rtol=1e-12, atol=1e-15) and slow == float(world))
            out.put(bool(ok))
    finally:
        dist.destroy_process_group()


def test_two_ranks_shard_rows_without_exchange_and_allreduce_dgain():
    ctx = mp.get_context("spawn")
    out = ctx.SimpleQueue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, 300, 256, out)) for r in range(2)]
    for p in procs:
        p.start()
    for p in procs:
        p.join(120)
        assert p.exitcode == 0
    assert out.get() is True
