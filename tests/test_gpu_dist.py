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
