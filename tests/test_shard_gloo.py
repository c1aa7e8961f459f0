"""N > 1: the batch is split across ranks with no data-path collective.  Two gloo ranks on the CPU check
the host-side logic: shard ranges tile the batch, per-sequence inputs do not depend on who generates them,
and the benchmark's max-over-ranks reduction."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import graft_inputs as gi
from paper_2608_20375_b200.shard import shard_range
from paper_2608_20375_b200.vocab_parallel import gather_partials, vocab_range


def test_shard_ranges_tile_the_batch():
    for batch in (0, 1, 7, 64, 65, 256):
        for world in (1, 2, 3, 8):
            spans = [shard_range(batch, r, world) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == batch
            assert all(a[1] == b[0] for a, b in zip(spans, spans[1:]))
            sizes = [hi - lo for lo, hi in spans]
            assert max(sizes) - min(sizes) <= 1


def _worker(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w = gi.small(batch=5, L=3, V=400, K=4)
    lo, hi = shard_range(w.batch, rank, world)
    x = gi.batch_inputs(w, lo, hi)
    digest = torch.tensor([float(x["logits"].double().sum()), float(hi - lo)], dtype=torch.float64)
    parts = [torch.zeros(2, dtype=torch.float64) for _ in range(world)]
    dist.all_gather(parts, digest)
    t = torch.tensor([1.0 + rank], dtype=torch.float64)  # stand-in for this rank's elapsed time
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    if rank == 0:
        q.put((torch.stack(parts).tolist(), float(t)))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_gloo():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    parts, tmax = q.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    w = gi.small(batch=5, L=3, V=400, K=4)
    full = gi.batch_inputs(w)
    assert abs(parts[0][0] + parts[1][0] - float(full["logits"].double().sum())) < 1e-6
    assert parts[0][1] + parts[1][1] == w.batch and tmax == 2.0


def test_vocab_ranges_tile_the_vocabulary():
    for V in (70, 9000, 32000, 151936):
        for world in (1, 2, 3, 5, 8):
            if V == 70 and world == 8:  # nine ids per rank cannot start on multiples of eight
                try:
                    vocab_range(V, 0, world)
                    assert False, "expected ValueError"
                except ValueError:
                    continue
            spans = [vocab_range(V, r, world) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == V and all(hi > lo for lo, hi in spans)
            assert all(a[1] == b[0] for a, b in zip(spans, spans[1:]))
            assert all(lo % 8 == 0 for lo, _ in spans)


def _gather_worker(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    rows = 6
    parts = torch.full((rows, 280), rank + 1, dtype=torch.uint8)  # stand-in for this rank's partial records
    parts[:, 0] = torch.arange(rows, dtype=torch.uint8)
    allp = gather_partials(parts)
    if rank == 1:
        q.put(allp.numpy().copy())
    dist.barrier()
    dist.destroy_process_group()


def test_partials_are_gathered_in_rank_order_gloo():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_gather_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    allp = q.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert allp.shape == (2, 6, 280)
    for r in range(2):
        assert (allp[r, :, 1:] == r + 1).all() and allp[r, :, 0].tolist() == list(range(6))
