"""World-size-2 checks of the rank plumbing on CPU (gloo): disjoint shares of independent
sequences reproduce the single-process result with no data-path exchange, and timing / throughput
reductions take the max / the sum over ranks."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2410_06577_b200 import dist as rdist
from paper_2410_06577_b200 import workloads as wl


def test_shard_units_partitions():
    for n in (0, 1, 7, 64, 65):
        for world in (1, 2, 3, 8):
            got = [i for r in range(world) for i in rdist.shard_units(n, r, world)]
            assert got == list(range(n))
            sizes = [len(rdist.shard_units(n, r, world)) for r in range(world)]
            assert max(sizes) - min(sizes) <= 1


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, out_dir):
    from oracle import ddts_oracle as orc
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank),
                      WORLD_SIZE=str(world), LOCAL_RANK=str(rank))
    r, w = rdist.init("gloo")
    assert (r, w) == (rank, world)
    cu = wl.varlen_lengths(9, 5, 3, 40)
    p = wl.make_prefill(9, 1, 2, int(cu[-1]), 8, 6, "f32", cu_seqlens=cu)
    mine = rdist.shard_units(5, rank, world)
    rows = slice(int(cu[mine.start]), int(cu[mine.stop]))
    sub_cu = (cu[mine.start:mine.stop + 1] - cu[mine.start]).astype(np.int32)
    sl = lambda a: np.ascontiguousarray(a[:, :, rows])
    o, sT = orc.ref_fwd(sl(p.q), sl(p.k), sl(p.x), sl(p.y), sl(p.v), cu_seqlens=sub_cu)
    np.save(os.path.join(out_dir, f"o{rank}.npy"), o)
    np.save(os.path.join(out_dir, f"s{rank}.npy"), sT)
    # reductions used by the benchmark
    assert rdist.max_over_ranks(10.0 + rank) == 10.0 + world - 1
    assert rdist.sum_over_ranks(float(len(mine))) == 5.0
    assert rdist.aggregate_throughput(100.0, 1.0 + rank) == pytest.approx(100.0 * world / world)
    rdist.barrier()
    dist.destroy_process_group()


def test_two_ranks_reproduce_single_process(tmp_path):
    from oracle import ddts_oracle as orc
    orc.build()
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    cu = wl.varlen_lengths(9, 5, 3, 40)
    p = wl.make_prefill(9, 1, 2, int(cu[-1]), 8, 6, "f32", cu_seqlens=cu)
    o, sT = orc.ref_fwd(p.q, p.k, p.x, p.y, p.v, cu_seqlens=cu)
    o_parts = [np.load(tmp_path / f"o{r}.npy") for r in range(world)]
    s_parts = [np.load(tmp_path / f"s{r}.npy") for r in range(world)]
    assert np.array_equal(np.concatenate(o_parts, axis=2), o)
    assert np.array_equal(np.concatenate(s_parts, axis=0), sT)
