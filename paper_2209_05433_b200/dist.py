"""Multi-GPU plumbing: one process per GPU over torch.distributed.

The hot path shards without a data-path collective when every rank owns whole
tensors (data-parallel replicas: each rank's activations and gradients are its
own, per-tensor amax is local).  When ONE tensor is split across ranks, its
per-tensor scale needs the maximum of the ranks' local amax values: a 4-byte
MAX all-reduce.  The amax travels as its binary32 bit pattern in an integer
tensor: magnitudes are non-negative, so integer order is value order, and the
canonical NaN pattern (0x7FC00000) sorts above infinity, which keeps the
reduction NaN-propagating and bit-exact for any rank count or order.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def shard_range(n: int, rank: int, world: int, align: int = 16) -> tuple[int, int]:
    """Contiguous [lo, hi) of a flat n-element tensor owned by `rank`; every boundary except the
    last is a multiple of `align` elements so that each shard keeps the 16-byte fast path."""
    if world < 1 or not 0 <= rank < world:
        raise ValueError("bad rank/world")
    units = -(-n // align)
    per = -(-units // world)
    lo = min(n, rank * per * align)
    hi = min(n, (rank + 1) * per * align)
    return lo, hi


def allreduce_amax_(amax: torch.Tensor, group=None) -> torch.Tensor:
    """In-place MAX all-reduce of a one-element float32 amax tensor (CPU with gloo, CUDA with NCCL)."""
    if amax.dtype != torch.float32 or amax.numel() != 1:
        raise TypeError("amax must be a one-element float32 tensor")
    bits = amax.view(torch.int32)
    dist.all_reduce(bits, op=dist.ReduceOp.MAX, group=group)
    return amax


def sharded_amax_scale_quantize(x_local: torch.Tensor, fmt: int, out_local: torch.Tensor, scratch: torch.Tensor, group=None):
    """Current scaling of a tensor split across ranks: local fp8_amax, 4-byte MAX all-reduce, the same
    scale on every rank, local fp8_quantize.  `scratch` is a 3-element float32 CUDA tensor that receives
    (amax, scale, scale_inv).  Every arithmetic step runs in the library's kernels."""
    from . import api
    a, s, si = scratch[0:1], scratch[1:2], scratch[2:3]
    api.fp8_amax(x_local, a)
    allreduce_amax_(a, group)
    api.fp8_scale_from_amax(a, fmt, s, si)
    api.fp8_quantize(x_local, fmt, s, out_local)
    return s, si


def column_shard(n_cols: int, rank: int, world: int) -> tuple[int, int]:
    """Columns [lo, hi) of a [rows, n_cols] weight or output owned by `rank`: boundaries are multiples of 16 columns,
    so that a shard of FP8 codes (1 byte per element) and of the bf16 / fp32 output both start on 16 bytes."""
    return shard_range(n_cols, rank, world, align=16)


def column_parallel_gemm(A, fmt_a, major_a, B_local, fmt_b, major_b, D_local, sa_inv, sb_inv, amax_d, group=None, **kw):
    """A product whose B operand (the weights of a forward layer) and output are split by output column across
    ranks: D[:, lo:hi] = A . B[:, lo:hi].  Every rank holds all of A and its own columns of B and D (views with the
    full row pitch are fine), so the contraction needs no exchange at all; the one per-tensor quantity of the whole
    output, the epilogue amax the next scale factor is chosen from, is the MAX over the ranks' amax values: the same
    4-byte all-reduce as for a sharded cast.  `amax_d` receives the amax of the WHOLE output on every rank."""
    from . import api
    api.fp8_gemm(A, fmt_a, major_a, B_local, fmt_b, major_b, D_local, sa_inv, sb_inv, amax_out=amax_d, **kw)
    allreduce_amax_(amax_d, group)
    return amax_d
