"""Every kernel of the library is deterministic (no atomics on data, fixed accumulation order), so repeated
launches on the same inputs must give bit-identical outputs.  A pipeline hazard (a shared-memory stage or a
TMEM accumulator reused too early, a store racing a barrier) shows up here as an occasional differing run
long before it shows up in a tolerance check."""
import pytest
import torch

from paper_2209_05433_b200 import api

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _codes(shape, gen):
    mag = torch.randint(0, 0x78, shape, dtype=torch.uint8, device=DEV, generator=gen)
    sign = torch.randint(0, 2, shape, dtype=torch.uint8, device=DEV, generator=gen) << 7
    return mag | sign


def _repeat(run, out, launches):
    run()
    torch.cuda.synchronize()
    ref = out.clone()
    differing = 0
    for i in range(launches):
        if i % 25 == 0:
            out.zero_()                     # a launch that silently skipped part of its output would show
        run()
        differing += int(not torch.equal(out.view(torch.uint8), ref.view(torch.uint8)))
    torch.cuda.synchronize()
    assert api.fp8_async_status()[0] == 0
    assert differing == 0, "%d of %d launches differ from the first" % (differing, launches)


@pytest.mark.parametrize("name,M,N,K,ma,mb", [("fprop", 8192, 16384, 4096, api.MAJOR_K, api.MAJOR_MN),
                                              ("dgrad", 8192, 4096, 16384, api.MAJOR_K, api.MAJOR_K),
                                              ("wgrad", 4096, 16384, 8192, api.MAJOR_MN, api.MAJOR_MN),
                                              ("ragged", 1000, 1300, 4208, api.MAJOR_K, api.MAJOR_K),
                                              ("short_k", 4096, 4096, 256, api.MAJOR_K, api.MAJOR_K)])
def test_gemm_is_bitwise_repeatable(name, M, N, K, ma, mb):
    gen = torch.Generator(device=DEV)
    gen.manual_seed(1)
    A = _codes((M, K) if ma == api.MAJOR_K else (K, M), gen)
    B = _codes((N, K) if mb == api.MAJOR_K else (K, N), gen)
    one = torch.ones(1, device=DEV)
    D = torch.empty(M, (N + 7) // 8 * 8, dtype=torch.bfloat16, device=DEV)[:, :N]
    D8 = torch.empty(M, (N + 15) // 16 * 16, dtype=torch.uint8, device=DEV)[:, :N]
    _repeat(lambda: api.fp8_gemm(A, api.E4M3, ma, B, api.E5M2, mb, D, one, one), D, 150)
    _repeat(lambda: api.fp8_gemm(A, api.E4M3, ma, B, api.E5M2, mb, D, one, one, acc=api.ACC_SPLIT), D, 100)
    _repeat(lambda: api.fp8_gemm_fp8out(A, api.E4M3, ma, B, api.E5M2, mb, D8, api.E4M3, one, one, one), D8, 100)


def test_batched_gemm_and_casts_are_bitwise_repeatable():
    gen = torch.Generator(device=DEV)
    gen.manual_seed(2)
    H, S, Dh = 16, 2048, 128
    Q, Kt = _codes((H, S, Dh), gen), _codes((H, S, Dh), gen)
    one = torch.ones(1, device=DEV)
    P = torch.empty(H, S, S, dtype=torch.bfloat16, device=DEV)
    _repeat(lambda: api.fp8_gemm_batched(Q, api.E4M3, api.MAJOR_K, Kt, api.E4M3, api.MAJOR_K, P, one, one), P, 150)
    x = torch.randn(4096, 8192, device=DEV, dtype=torch.bfloat16, generator=gen)
    o = torch.empty(4096, 8192, dtype=torch.uint8, device=DEV)
    ot = torch.empty(8192, 4096, dtype=torch.uint8, device=DEV)
    s3, sc = torch.full((1,), 3.0, device=DEV), torch.zeros(3, device=DEV)
    _repeat(lambda: api.fp8_quantize_transpose(x, api.E4M3, s3, o, ot, sc[0:1]), ot, 150)
    _repeat(lambda: api.fp8_quantize_current(x, api.E5M2, o, sc[0:1], sc[1:2], sc[2:3]), o, 150)
    back = torch.empty_like(x)
    _repeat(lambda: api.fp8_fake_quantize(x, api.E4M3, s3, sc[2:3], back), back, 100)


def test_back_to_back_dependent_casts_see_each_others_results():
    """The cast kernels are launched with programmatic stream serialization (a kernel may be scheduled while its
    predecessor drains).  Chains in which every kernel consumes what the one before it wrote, enqueued without any
    host synchronisation and with buffers that are overwritten from one round to the next, must give the results of
    strictly serial execution: codes -> dequantize equals the one-pass simulated conversion, round after round."""
    import numpy as np
    from paper_2209_05433_b200 import synth
    dev = "cuda"
    sizes = [(1 << 12) + 8, 1 << 16, (1 << 20) + 16, 1 << 22, (1 << 23) + 24]
    xs = [synth.normal_laplace_mixture(n, 31 + i, synth.T_ID, dtype=torch.bfloat16, device=dev) for i, n in enumerate(sizes)]
    nmax = max(sizes)
    codes = torch.empty(nmax, dtype=torch.uint8, device=dev)          # shared scratch, rewritten by every round
    back = torch.empty(nmax, dtype=torch.bfloat16, device=dev)
    direct = torch.empty(nmax, dtype=torch.bfloat16, device=dev)
    sc = torch.zeros(3, dtype=torch.float32, device=dev)
    a, s, si = sc[0:1], sc[1:2], sc[2:3]
    bad = torch.zeros(1, dtype=torch.int64, device=dev)
    for rnd in range(40):
        for x in xs:
            n = x.numel()
            fmt = api.E4M3 if rnd & 1 else api.E5M2
            api.fp8_amax(x, a)                                        # zeroing kernel + reduction
            api.fp8_scale_from_amax(a, fmt, s, si)                    # reads the amax
            api.fp8_quantize(x, fmt, s, codes[:n])                    # reads the scale
            api.fp8_dequantize(codes[:n], fmt, si, back[:n])          # reads the codes and the inverse scale
            api.fp8_fake_quantize(x, fmt, s, si, direct[:n])          # the same arithmetic in one pass
            bad += (back[:n].view(torch.int16) != direct[:n].view(torch.int16)).sum()
    torch.cuda.synchronize()
    assert api.fp8_async_status()[0] == 0
    assert int(bad.item()) == 0
