"""Full-size workloads (transformer linear layers at hidden 4096 and 12288), run in the launch
configuration the benchmark times, checked against the CPU oracle on samples it can compute one by one:
 - scales: the oracle's amax of the WHOLE tensor and its scale arithmetic, bit-exact;
 - codes: first and last 2^20 elements plus random 64Ki blocks, bit-exact;
 - GEMM outputs: the first and the last row in full, one interior 256 x 256 output tile (the unit one CTA pair
   computes) and the last one in full (every fourth row where K = 49152), the four corners of random output
   tiles, and 2^20 random (i, j) at hidden 4096 / 2^16 at hidden 12288, each against the fp64 dot product of
   the decoded operands;
 - epilogue amax: equal to the library's amax of D as stored, and to the oracle's amax of the stored D.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2209_05433_b200 import api, synth
from tests._util import THREADS, check_gemm_bf16, to_np_bits

pytestmark = pytest.mark.gpu
DEV = "cuda"
E4, E5 = oracle.E4M3, oracle.E5M2


def _scalar():
    return torch.zeros(1, dtype=torch.float32, device=DEV)


def _cast(x, fmt, rng):
    """current scaling through the library, as three calls and as the one launch the benchmark times; verified
    against the oracle; returns (codes, scale_inv, host codes, oracle's scale_inv)"""
    n = x.numel()
    a, s, si = _scalar(), _scalar(), _scalar()
    codes = torch.empty(n, dtype=torch.uint8, device=DEV)
    api.fp8_amax(x, a)
    api.fp8_scale_from_amax(a, fmt, s, si)
    api.fp8_quantize(x.view(-1), fmt, s, codes)
    torch.cuda.synchronize()
    x_host = to_np_bits(x.view(-1))
    ws, wsi = oracle.scale_from_amax(oracle.amax(x_host, THREADS), fmt)
    assert s.item() == ws and si.item() == wsi
    codes_host = codes.cpu().numpy()
    blk = 1 << 20
    blocks = [(0, min(n, blk)), (max(0, n - blk), n)] + [(int(b) << 16, (int(b) + 1) << 16) for b in rng.integers(0, n >> 16, size=16)]
    for lo, hi in blocks:
        want = oracle.quantize(x_host[lo:hi], ws, fmt, threads=THREADS)
        assert np.array_equal(codes_host[lo:hi], want), (lo, hi)
    # the one-launch form the benchmark step uses: same amax, scales and codes, everywhere
    a1, s1, si1 = _scalar(), _scalar(), _scalar()
    codes1 = torch.empty(n, dtype=torch.uint8, device=DEV)
    api.fp8_quantize_current(x.view(-1), fmt, codes1, a1, s1, si1)
    torch.cuda.synchronize()
    assert api.fp8_async_status()[0] == 0
    assert a1.item() == a.item() and s1.item() == ws and si1.item() == wsi
    assert torch.equal(codes1, codes)
    return codes, si, codes_host, wsi


def _sample_positions(M, N, rng, n_random, tile_row_step, n_tiles=64):
    ii = [np.zeros(N, dtype=np.int64), np.full(N, M - 1, dtype=np.int64)]
    jj = [np.arange(N, dtype=np.int64), np.arange(N, dtype=np.int64)]
    # two whole output tiles of the kernel (256 x 256, one CTA pair each): one in the interior, and the last one
    tiles_m, tiles_n = (M + 255) // 256, (N + 255) // 256
    for tm_, tn_ in ((tiles_m // 2, tiles_n // 2 + 1 if tiles_n > 2 else 0), (tiles_m - 1, tiles_n - 1)):
        r = np.arange(tm_ * 256, min(M, tm_ * 256 + 256), tile_row_step, dtype=np.int64)
        c = np.arange(tn_ * 256, min(N, tn_ * 256 + 256), dtype=np.int64)
        gi, gj = np.meshgrid(r, c, indexing="ij")
        ii.append(gi.ravel())
        jj.append(gj.ravel())
    tm = rng.integers(0, (M + 127) // 128, size=n_tiles)
    tn = rng.integers(0, (N + 255) // 256, size=n_tiles)
    for di in (0, 127):
        for dj in (0, 255):
            ii.append(np.minimum(tm * 128 + di, M - 1))
            jj.append(np.minimum(tn * 256 + dj, N - 1))
    ii.append(rng.integers(0, M, size=n_random))
    jj.append(rng.integers(0, N, size=n_random))
    return np.concatenate(ii), np.concatenate(jj)


LITERAL = {}      # label -> fraction of sampled outputs within 1 bf16 ulp of the correctly rounded reference


def _check_gemm(D, amax, A_host, fa, a_str, B_host, fb, b_str, K, sa_inv, sb_inv, rng, label, n_random, tile_row_step=1):
    torch.cuda.synchronize()
    st, detail = api.fp8_async_status()
    assert st == 0, "device-side wait expired, code %d" % detail
    M, N = D.shape
    ii, jj = _sample_positions(M, N, rng, n_random, tile_row_step)
    ref, sabs = oracle.gemm_samples(A_host, fa, a_str, B_host, fb, b_str, K, ii, jj, sa_inv, sb_inv, threads=THREADS)
    got = to_np_bits(D[torch.from_numpy(ii).to(DEV), torch.from_numpy(jj).to(DEV)])
    ok, literal = check_gemm_bf16(got, ref, sabs, oracle.round_bf16_from_f64)
    assert ok.all(), "%s: %d of %d sampled outputs out of tolerance, first at %s" % (
        label, (~ok).sum(), ok.size, [(int(ii[k]), int(jj[k])) for k in np.nonzero(~ok)[0][:4]])
    a2 = _scalar()
    api.fp8_amax(D, a2)
    bits = amax.cpu().numpy().view(np.uint32)[0]
    assert bits == a2.cpu().numpy().view(np.uint32)[0]
    assert bits == oracle.amax_bits(to_np_bits(D).reshape(-1), THREADS)
    LITERAL[label] = (float(literal.mean()), int(literal.size))
    print("%s: %d sampled outputs, %.6f within 1 bf16 ulp of the rounded reference" % (label, literal.size, literal.mean()))
    # zero-mean operands: cancellation is rare, so nearly every output meets the literal test as well
    assert literal.mean() > 0.999, (label, literal.mean())


def _linear_layer(seed, T, I, O, w_sigma, passes, n_random):
    rng = np.random.default_rng(seed)
    X = synth.activations(T * I, seed, device=DEV).view(T, I)
    W = synth.weights(I * O, seed, w_sigma, device=DEV).view(I, O)
    Xq, six, Xh, wsix = _cast(X, api.E4M3, rng)
    Wq, siw, Wh, wsiw = _cast(W, api.E4M3, rng)
    del X, W
    Xq, Wq = Xq.view(T, I), Wq.view(I, O)
    amax = _scalar()
    if "fprop" in passes:        # Y[T,O] = X[T,I] . W[I,O]
        Y = torch.empty(T, O, dtype=torch.bfloat16, device=DEV)
        api.fp8_gemm(Xq, api.E4M3, api.MAJOR_K, Wq, api.E4M3, api.MAJOR_MN, Y, six, siw, amax)
        _check_gemm(Y, amax, Xh, E4, (I, 1), Wh, E4, (O, 1), I, wsix, wsiw, rng, "fprop K=%d" % I, n_random)
        # the same product with one accumulator over all of K (FP8_ACC_FAST; the default adds partial sums every 2048 of K)
        api.fp8_gemm(Xq, api.E4M3, api.MAJOR_K, Wq, api.E4M3, api.MAJOR_MN, Y, six, siw, amax, acc=api.ACC_FAST)
        _check_gemm(Y, amax, Xh, E4, (I, 1), Wh, E4, (O, 1), I, wsix, wsiw, rng, "fprop K=%d one accumulator" % I, n_random // 8, 4)
        del Y
    if "dgrad" in passes or "wgrad" in passes:
        dY = synth.gradients(T * O, seed, device=DEV).view(T, O)
        Gq, sig, Gh, wsig = _cast(dY, api.E5M2, rng)
        del dY
        Gq = Gq.view(T, O)
        if "dgrad" in passes:    # dX[T,I] = dY[T,O] . W^T
            dX = torch.empty(T, I, dtype=torch.bfloat16, device=DEV)
            api.fp8_gemm(Gq, api.E5M2, api.MAJOR_K, Wq, api.E4M3, api.MAJOR_K, dX, sig, siw, amax)
            step = 4 if O > 16384 else 1                  # K = 49152: every fourth row of the two whole tiles
            _check_gemm(dX, amax, Gh, E5, (O, 1), Wh, E4, (1, O), O, wsig, wsiw, rng, "dgrad K=%d" % O, n_random, step)
            # the same product with one accumulator over all of K (FP8_ACC_FAST; the default adds partial sums every 2048 of K)
            api.fp8_gemm(Gq, api.E5M2, api.MAJOR_K, Wq, api.E4M3, api.MAJOR_K, dX, sig, siw, amax, acc=api.ACC_FAST)
            _check_gemm(dX, amax, Gh, E5, (O, 1), Wh, E4, (1, O), O, wsig, wsiw, rng, "dgrad K=%d one accumulator" % O, n_random // 4, 4 * step)
            del dX
        if "wgrad" in passes:    # dW[I,O] = X^T . dY
            dW = torch.empty(I, O, dtype=torch.bfloat16, device=DEV)
            api.fp8_gemm(Xq, api.E4M3, api.MAJOR_MN, Gq, api.E5M2, api.MAJOR_MN, dW, six, sig, amax)
            _check_gemm(dW, amax, Xh, E4, (1, I), Gh, E5, (O, 1), T, wsix, wsig, rng, "wgrad K=%d" % T, n_random)
            api.fp8_gemm(Xq, api.E4M3, api.MAJOR_MN, Gq, api.E5M2, api.MAJOR_MN, dW, six, sig, amax, acc=api.ACC_FAST)
            _check_gemm(dW, amax, Xh, E4, (1, I), Gh, E5, (O, 1), T, wsix, wsig, rng, "wgrad K=%d one accumulator" % T, n_random // 8, 4)
            del dW
    torch.cuda.empty_cache()


def test_config3_forward_linear_hidden_4096():
    """activations [8192 x 4096] N(0,1) + 0.1% outliers of magnitude 20-100, weights [4096 x 16384] N(0,0.02),
    both to E4M3; forward GEMM M=8192 N=16384 K=4096, bf16 out with epilogue amax"""
    _linear_layer(3, 8192, 4096, 16384, 0.02, ("fprop",), 1 << 20)


def test_config4_backward_hidden_4096():
    """output gradients [8192 x 16384] 1e-4 * Student-t(3) to E5M2; dgrad M=8192 N=4096 K=16384 and
    wgrad M=4096 N=16384 K=8192, bf16 out"""
    _linear_layer(4, 8192, 4096, 16384, 0.02, ("dgrad", "wgrad"), 1 << 20)


def test_config5_ffn_hidden_12288():
    """175B-class FFN: activations [8192 x 12288], weights [12288 x 49152] N(0,0.006); forward GEMM
    M=8192 N=49152 K=12288 and the E5M2-gradient dgrad GEMM M=8192 N=12288 K=49152"""
    _linear_layer(5, 8192, 12288, 49152, 0.006, ("fprop", "dgrad"), 1 << 16)
