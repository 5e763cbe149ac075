"""The sharded current-scaling path on the GPU: one tensor split across two ranks, each rank running the
library's own kernels on its shard (fp8_amax -> 4-byte MAX all-reduce -> fp8_scale_from_amax -> fp8_quantize).

Two gloo ranks share the one GPU of the test box (CUDA tensors, host-staged all-reduce).  No kernel of one
rank waits for a kernel of the other: each rank's launches are ordinary stream work, and the only exchange is
the all-reduce of the 4-byte amax, which the ranks enter from the host.  Checked against the oracle's codes of
the WHOLE tensor, with the maximum (or a NaN) sitting in the second shard."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

pytestmark = pytest.mark.gpu


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, n, special, fmt, ret):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        import oracle
        from paper_2209_05433_b200 import api, synth
        from paper_2209_05433_b200 import dist as fdist
        torch.cuda.set_device(0)
        x = synth.activations(n, 21, dtype=torch.bfloat16)              # the whole tensor, identical on both ranks (host)
        if special == "max":
            x[n - 7] = 3000.0                                           # the maximum lives in the last rank's shard
        elif special == "nan":
            x[n - 7] = float("nan")
        lo, hi = fdist.shard_range(n, rank, world)
        x_local = x[lo:hi].cuda()
        out_local = torch.empty(hi - lo, dtype=torch.uint8, device="cuda")
        scratch = torch.zeros(3, dtype=torch.float32, device="cuda")
        s, si = fdist.sharded_amax_scale_quantize(x_local, fmt, out_local, scratch)
        torch.cuda.synchronize()
        assert api.fp8_async_status() == (0, 0)
        bits = x.view(torch.int16).numpy().view(np.uint16)
        want_amax = oracle.amax(bits)
        ws, wsi = oracle.scale_from_amax(want_amax, fmt)
        whole = oracle.quantize(bits, ws, fmt)
        got_amax = scratch[0:1].cpu().numpy().view(np.uint32)[0]
        ret[rank] = (int(got_amax) == int(np.array([want_amax]).view(np.uint32)[0]), float(s.item()) == float(ws),
                     float(si.item()) == float(wsi), bool(np.array_equal(out_local.cpu().numpy(), whole[lo:hi])), (lo, hi))
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("special", ["max", "nan"])
@pytest.mark.parametrize("fmt", [0, 1])
def test_two_ranks_quantize_one_tensor_with_one_scale(special, fmt):
    world, n = 2, (1 << 20) + 1003
    port = _free_port()
    manager = mp.Manager()
    ret = manager.dict()
    mp.spawn(_worker, args=(world, port, n, special, fmt, ret), nprocs=world, join=True)
    assert len(ret) == world
    for rank in range(world):
        same_amax, same_scale, same_inv, same_codes, _ = ret[rank]
        assert same_amax and same_scale and same_inv and same_codes, (rank, ret[rank])
    assert ret[0][4][1] == ret[1][4][0] and ret[0][4][0] == 0 and ret[1][4][1] == n


def _worker_columns(rank, world, port, ret):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        import oracle
        from paper_2209_05433_b200 import api, synth
        from paper_2209_05433_b200 import dist as fdist
        from tests._util import THREADS, check_gemm_bf16, to_np_bits
        torch.cuda.set_device(0)
        T, I, O = 384, 2304, 1008                                        # K spans two 2048-chunks; O is not a multiple of the tile
        X = synth.activations(T * I, 31, dtype=torch.bfloat16).view(T, I)
        W = synth.weights(I * O, 32, 0.02, dtype=torch.bfloat16).view(I, O)
        W[5, O - 3] = 40.0                                               # the largest output sits in the last rank's columns
        xb, wb = to_np_bits(X).reshape(-1), to_np_bits(W).reshape(-1)
        sx, six = oracle.scale_from_amax(oracle.amax(xb), oracle.E4M3)
        sw, siw = oracle.scale_from_amax(oracle.amax(wb), oracle.E4M3)
        Xq = oracle.quantize(xb, sx, oracle.E4M3).reshape(T, I)
        Wq = oracle.quantize(wb, sw, oracle.E4M3).reshape(I, O)
        lo, hi = fdist.column_shard(O, rank, world)
        Xd, Wd = torch.from_numpy(Xq).cuda(), torch.from_numpy(Wq).cuda()          # every rank holds the whole tensors here; it
        Y = torch.zeros(T, O, dtype=torch.bfloat16, device="cuda")                  # touches only its own columns of W and Y
        sc = torch.tensor([six, siw, 0.0], dtype=torch.float32, device="cuda")
        fdist.column_parallel_gemm(Xd, api.E4M3, api.MAJOR_K, Wd[:, lo:hi], api.E4M3, api.MAJOR_MN, Y[:, lo:hi], sc[0:1], sc[1:2], sc[2:3])
        torch.cuda.synchronize()
        assert api.fp8_async_status() == (0, 0)
        ref, sab = oracle.gemm_rows(Xq, oracle.E4M3, (I, 1), Wq, oracle.E4M3, (O, 1), O, I, 0, T, six, siw, threads=THREADS)
        got = to_np_bits(Y).reshape(T, O)
        ok, _ = check_gemm_bf16(got[:, lo:hi], ref[:, lo:hi], sab[:, lo:hi], oracle.round_bf16_from_f64)
        untouched = bool((np.delete(got, np.s_[lo:hi], axis=1) == 0).all())
        # amax of the WHOLE output as stored: the other rank's columns are rounded from the oracle's reference (the two
        # may differ by the accumulation tolerance, so compare with a tolerance of one bf16 step of the maximum)
        whole = oracle.round_bf16_from_f64(ref).astype(np.uint16).reshape(T, O).copy()
        whole[:, lo:hi] = got[:, lo:hi]
        want = int(((whole & 0x7FFF).max()).astype(np.uint32)) << 16
        got_amax = int(sc[2:3].cpu().numpy().view(np.uint32)[0])
        ret[rank] = (bool(ok.all()), untouched, abs(got_amax - want) <= (1 << 16), got_amax, (lo, hi))
    finally:
        dist.destroy_process_group()


def test_two_ranks_split_the_output_columns_of_a_forward_product():
    """column-parallel forward product: no exchange in the contraction, one 4-byte MAX all-reduce for the amax"""
    world = 2
    port = _free_port()
    manager = mp.Manager()
    ret = manager.dict()
    mp.spawn(_worker_columns, args=(world, port, ret), nprocs=world, join=True)
    assert len(ret) == world
    for rank in range(world):
        in_tolerance, untouched, amax_ok, _, _ = ret[rank]
        assert in_tolerance and untouched and amax_ok, (rank, ret[rank])
    assert ret[0][3] == ret[1][3]                                        # every rank ends with the same amax
    assert ret[0][4][0] == 0 and ret[0][4][1] == ret[1][4][0] and ret[1][4][1] == 1008 and ret[0][4][1] % 16 == 0
