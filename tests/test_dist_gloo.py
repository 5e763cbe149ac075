"""world_size-2 gloo test (CPU) of the multi-GPU host logic: contiguous aligned sharding and the
bit-pattern MAX all-reduce of amax.  Local amax values come from the oracle here (no GPU); the point is
that shards + reduction reproduce the whole-tensor amax and scale bit for bit, NaN included."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
from paper_2209_05433_b200 import dist as fdist


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, n, with_nan, ret):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        rng = np.random.default_rng(123)
        x = (rng.standard_normal(n) * np.exp2(rng.uniform(-8, 8, size=n))).astype(np.float32)
        if with_nan:
            x[n - 3] = np.nan                          # lives in the last rank's shard
        lo, hi = fdist.shard_range(n, rank, world)
        local_bits = oracle.amax_bits(x[lo:hi])
        amax = torch.from_numpy(np.array([local_bits], dtype=np.uint32).view(np.float32).copy())
        fdist.allreduce_amax_(amax)
        got_bits = int(amax.numpy().view(np.uint32)[0])
        want_bits = oracle.amax_bits(x)
        scale = oracle.scale_from_amax(amax.numpy()[0], oracle.E4M3)
        want_scale = oracle.scale_from_amax(np.array([want_bits], dtype=np.uint32).view(np.float32)[0], oracle.E4M3)
        # quantizing the shard with the reduced scale equals the shard of the whole-tensor result
        codes = oracle.quantize(x[lo:hi], scale[0], oracle.E4M3)
        whole = oracle.quantize(x, want_scale[0], oracle.E4M3)
        ret[rank] = (got_bits == want_bits, scale == want_scale, bool(np.array_equal(codes, whole[lo:hi])), (lo, hi))
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("with_nan", [False, True])
def test_two_rank_amax_allreduce_matches_whole_tensor(with_nan):
    world, n = 2, 100003
    port = _free_port()
    manager = mp.Manager()
    ret = manager.dict()
    mp.spawn(_worker, args=(world, port, n, with_nan, ret), nprocs=world, join=True)
    assert len(ret) == world
    for rank in range(world):
        same_amax, same_scale, same_codes, _ = ret[rank]
        assert same_amax and same_scale and same_codes
    assert ret[0][3][1] == ret[1][3][0] and ret[0][3][0] == 0 and ret[1][3][1] == n


def test_shard_range_partitions_exactly():
    for n in (0, 1, 15, 16, 17, 1000, 100003, 1 << 20):
        for world in (1, 2, 3, 8):
            spans = [fdist.shard_range(n, r, world) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == n
            for (a, b), (c, d) in zip(spans[:-1], spans[1:]):
                assert b == c and a <= b and (b % 16 == 0 or b == n)


def test_column_shards_partition_the_output_columns_on_16_byte_boundaries():
    for cols in (16, 1008, 4096, 49152, 12345):
        for world in (1, 2, 3, 8):
            spans = [fdist.column_shard(cols, r, world) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == cols
            for (a, b), (c, d) in zip(spans[:-1], spans[1:]):
                assert b == c and a <= b and (b % 16 == 0 or b == cols)
