"""World-size-2 check (gloo, CPU) of the multi-rank host logic: units are split without overlap or gap,
every rank encodes and validates its own share, and only byte counts and timings are reduced - the same
reductions bench.py performs over NCCL."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2609_34185_b200.sharding import shard_range, tile_range_rows


def test_shard_range_partitions():
    for n in (0, 1, 7, 48, 4610):
        for world in (1, 2, 3, 8):
            got = [i for r in range(world) for i in shard_range(n, world, r)]
            assert got == list(range(n))
            sizes = [len(shard_range(n, world, r)) for r in range(world)]
            assert max(sizes) - min(sizes) <= 1


def _worker(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import oracle
    import paper_2609_34185_b200 as ep
    from paper_2609_34185_b200 import synth
    shapes = [(64, 512), (32, 1024), (96, 256), (48, 768), (16, 2048)]
    mine = shard_range(len(shapes), world, rank)
    nbytes, params = 0, 0
    for i in mine:
        W = synth.gaussian_rows(*shapes[i], seed=900 + i)
        blob = ep.encode(W, 4.0, tile_vectors=64, threads=2)
        assert ep.validate(blob.data) == 0
        out, _ = oracle.decode(blob.data, oracle.BF16)          # CPU stand-in for the rank's GPU decode
        assert out.shape == shapes[i]
        r0, r1 = tile_range_rows(blob.info, shard_range(blob.info.n_tiles, 2, 1))
        assert 0 <= r0 < r1 <= shapes[i][0]
        nbytes += len(blob)
        params += W.size
    # one tensor split by tile ranges (the shard of a tensor-parallel rank): the ranks' ranges are disjoint and
    # cover the tensor, so the sum of their zero-filled partial decodes is the full decode
    Wt = synth.laplace_rows(48, 512, 950)
    bt = ep.encode(Wt, 3.0, tile_vectors=100, threads=2)
    tiles = shard_range(bt.info.n_tiles, world, rank)
    part, _ = oracle.decode(bt.data, oracle.BF16, tiles=(tiles.start, tiles.stop))
    acc = torch.from_numpy(part.astype(np.int64))
    dist.all_reduce(acc)                                         # test-only: the product path exchanges nothing
    full, _ = oracle.decode(bt.data, oracle.BF16)
    assert np.array_equal(acc.numpy(), full.astype(np.int64))
    t = torch.tensor([float(nbytes), float(params)], dtype=torch.float64)
    dist.all_reduce(t)                                           # whole-job totals
    tm = torch.tensor([1.0 + rank], dtype=torch.float64)
    dist.all_reduce(tm, op=dist.ReduceOp.MAX)                    # max-over-ranks timing
    dist.barrier()
    if rank == 0:
        q.put((t.tolist(), tm.item(), list(mine)))
    dist.destroy_process_group()


def test_two_ranks_cover_all_units_without_a_collective_on_the_data_path():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    totals, tmax, mine0 = q.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert totals[1] == float(64 * 512 + 32 * 1024 + 96 * 256 + 48 * 768 + 16 * 2048)
    assert abs(8 * totals[0] / totals[1] - 4.0) < 0.6          # tiny tensors with 64-vector tiles: metadata-heavy
    assert tmax == 2.0 and mine0 == [0, 1]
