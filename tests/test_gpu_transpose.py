"""GPU parity of fp8_quantize_transpose against the CPU oracle: the codes are the oracle's quantize of every
element (bit-exact), stored row-major and as the transposed matrix; amax is the oracle's amax of x.
Everything goes through the C ABI (paper_2209_05433_b200.api)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2209_05433_b200 import api, synth
from tests._util import THREADS, to_np_bits

pytestmark = pytest.mark.gpu

DEV = "cuda"
FMTS = [oracle.E4M3, oracle.E5M2]
GUARD = 0xA5


def _scalar(v):
    return torch.tensor([v], dtype=torch.float32, device=DEV)


def _run(x, fmt, scale, overflow=api.SATURATE, pad_o=0, pad_t=0, with_out=True, with_amax=True):
    """x: 2-D device tensor (any pitch).  Returns (out or None, out_t, amax bits or None) as numpy, after
    checking that nothing outside the logical extents was written."""
    rows, cols = x.shape
    out_full = torch.full((rows + 1, cols + pad_o), GUARD, dtype=torch.uint8, device=DEV)
    t_full = torch.full((cols + 1, rows + pad_t), GUARD, dtype=torch.uint8, device=DEV)
    out = out_full[:rows, :cols] if with_out else None
    out_t = t_full[:cols, :rows]
    amax = _scalar(-1.0) if with_amax else None
    api.fp8_quantize_transpose(x, fmt, _scalar(scale), out, out_t, amax, overflow)
    torch.cuda.synchronize()
    assert bool((t_full[cols:, :] == GUARD).all()) and bool((t_full[:cols, rows:] == GUARD).all()), "wrote outside out_t"
    if with_out:
        assert bool((out_full[rows:, :] == GUARD).all()) and bool((out_full[:rows, cols:] == GUARD).all()), "wrote outside out"
    else:
        assert bool((out_full == GUARD).all())
    return (out.cpu().numpy() if with_out else None, out_t.cpu().numpy(),
            amax.cpu().numpy().view(np.uint32)[0] if with_amax else None)


def _check(x, fmt, scale, overflow=api.SATURATE, **kw):
    rows, cols = x.shape
    xb = to_np_bits(x)                         # contiguous copy of the logical matrix
    want = oracle.quantize(xb.reshape(-1), np.float32(scale), fmt, overflow, threads=THREADS).reshape(rows, cols)
    out, out_t, bits = _run(x, fmt, scale, overflow, **kw)
    if out is not None:
        bad = np.argwhere(out != want)
        assert bad.size == 0, "row-major: %d mismatches, first %s" % (len(bad), bad[:4].tolist())
    bad = np.argwhere(out_t != want.T)
    assert bad.size == 0, "transposed: %d mismatches, first %s" % (len(bad), bad[:4].tolist())
    if bits is not None:
        assert bits == oracle.amax_bits(xb.reshape(-1), THREADS)


def _random(rows, cols, wide, seed, pitch_pad=0):
    n = rows * (cols + pitch_pad)
    x = synth.normal_laplace_mixture(n, seed, synth.T_ID, device=DEV)
    if wide == torch.float32:
        x = x.float() * 1.00390625            # values that are not bf16-representable
    return x.view(rows, cols + pitch_pad)[:, :cols]


@pytest.mark.parametrize("wide", [torch.bfloat16, torch.float32])
@pytest.mark.parametrize("fmt", FMTS)
@pytest.mark.parametrize("rows,cols", [(128, 128), (256, 384), (4, 4), (132, 260), (1024, 36), (8, 1028), (640, 1152)])
def test_tiled_path_shapes(wide, fmt, rows, cols):
    """multiples of 4 in both extents: whole tiles, ragged tiles on either edge, a single 4 x 4 block"""
    x = _random(rows, cols, wide, rows + cols)
    _check(x, fmt, 37.5)


@pytest.mark.parametrize("wide", [torch.bfloat16, torch.float32])
@pytest.mark.parametrize("rows,cols,pitch_pad,pad_o,pad_t", [(256, 256, 4, 4, 4), (132, 260, 12, 8, 20), (128, 384, 0, 0, 4)])
def test_tiled_path_pitches(wide, rows, cols, pitch_pad, pad_o, pad_t):
    """row pitches larger than the rows (multiples of 4), for the input and for both outputs"""
    x = _random(rows, cols, wide, 7, pitch_pad)
    _check(x, oracle.E4M3, 12.0, pad_o=pad_o, pad_t=pad_t)


@pytest.mark.parametrize("wide", [torch.bfloat16, torch.float32])
@pytest.mark.parametrize("rows,cols,pitch_pad,pad_o,pad_t", [(130, 67, 0, 0, 0), (1, 1, 0, 0, 0), (3, 500, 1, 0, 0), (257, 129, 3, 5, 7),
                                                             (128, 128, 1, 0, 0), (128, 128, 0, 1, 0), (128, 128, 0, 0, 2)])
def test_elementwise_path(wide, rows, cols, pitch_pad, pad_o, pad_t):
    """extents or pitches that are not multiples of 4: identical results from the element-wise kernel"""
    x = _random(rows, cols, wide, 11, pitch_pad)
    _check(x, oracle.E5M2, 3.0, pad_o=pad_o, pad_t=pad_t)


def test_unaligned_base_pointers():
    base = synth.normal_laplace_mixture(256 * 256 + 8, 5, synth.T_ID, device=DEV)
    for off in (1, 2, 3, 4):
        x = base[off: off + 256 * 256].view(256, 256)
        _check(x, oracle.E4M3, 5.0)


@pytest.mark.parametrize("wide", [torch.bfloat16, torch.float32])
@pytest.mark.parametrize("fmt", FMTS)
@pytest.mark.parametrize("overflow", [api.SATURATE, api.NOSAT])
def test_special_values_and_overflow_modes(wide, fmt, overflow):
    """NaN of both signs, infinities, zeros of both signs, values around the overflow thresholds, and a scale
    that pushes finite inputs to infinity: the scalar encoder takes over for any group of four that holds one"""
    rows, cols = 256, 384
    x = _random(rows, cols, wide, 3).clone()
    specials = [float("nan"), -float("nan"), float("inf"), -float("inf"), 0.0, -0.0, 448.0, 464.0, 465.0, 480.0,
                57344.0, 61439.0, 61440.0, -61440.0, 3.0e38, -3.0e38, 2.0 ** -9, 2.0 ** -10, 2.0 ** -17, 1.0e-40]
    rng = np.random.default_rng(9)
    flat = x.view(-1) if x.is_contiguous() else None
    assert flat is not None
    idx = torch.from_numpy(rng.choice(rows * cols, size=40 * len(specials), replace=False)).to(DEV)
    vals = torch.tensor(specials * 40, dtype=torch.float32, device=DEV).to(wide)
    flat[idx] = vals
    neg_nan = torch.tensor([0xFFC0], dtype=torch.uint16).view(torch.bfloat16).to(DEV)
    flat[idx[1::len(specials)]] = neg_nan.to(wide) if wide == torch.bfloat16 else torch.tensor([0xFFC00000], dtype=torch.uint32).view(torch.float32).to(DEV)
    for scale in (1.0, 2.0, 1.0e3):
        _check(x, fmt, scale, overflow)


@pytest.mark.parametrize("fmt", FMTS)
def test_transposed_only_and_no_amax(fmt):
    x = _random(384, 256, torch.bfloat16, 21)
    _check(x, fmt, 9.0, with_out=False, with_amax=False)
    _check(x, fmt, 9.0, with_out=False, with_amax=True)
    _check(x, fmt, 9.0, with_out=True, with_amax=False)


def test_empty_and_amax_reset():
    amax = _scalar(5.0)
    x = torch.empty((0, 16), dtype=torch.bfloat16, device=DEV)
    api.fp8_quantize_transpose(x, api.E4M3, _scalar(1.0), torch.empty((0, 16), dtype=torch.uint8, device=DEV),
                               torch.empty((16, 0), dtype=torch.uint8, device=DEV), amax)
    assert amax.item() == 0.0


def test_equals_quantize_and_feeds_the_weight_gradient_gemm():
    """the transposed codes are K-major operands of the weight-gradient product dW = X^T . dY: the GEMM on them
    equals, bit for bit, the GEMM on the row-major codes read MN-major"""
    T, I, O = 512, 384, 640
    X = synth.activations(T * I, 1, device=DEV).view(T, I)
    dY = synth.gradients(T * O, 1, device=DEV).view(T, O)
    sx, sg = _scalar(2.0), _scalar(4096.0)
    Xq, XqT = torch.empty(T, I, dtype=torch.uint8, device=DEV), torch.empty(I, T, dtype=torch.uint8, device=DEV)
    Gq, GqT = torch.empty(T, O, dtype=torch.uint8, device=DEV), torch.empty(O, T, dtype=torch.uint8, device=DEV)
    api.fp8_quantize_transpose(X, api.E4M3, sx, Xq, XqT)
    api.fp8_quantize_transpose(dY, api.E5M2, sg, Gq, GqT)
    ref = torch.empty(T * I, dtype=torch.uint8, device=DEV)
    api.fp8_quantize(X.view(-1), api.E4M3, sx, ref)
    assert torch.equal(ref.view(T, I), Xq) and torch.equal(Xq.t().contiguous(), XqT)
    si_x, si_g = _scalar(0.5), _scalar(1.0 / 4096.0)
    dW0 = torch.empty(I, O, dtype=torch.float32, device=DEV)
    dW1 = torch.empty_like(dW0)
    api.fp8_gemm(Xq, api.E4M3, api.MAJOR_MN, Gq, api.E5M2, api.MAJOR_MN, dW0, si_x, si_g)
    api.fp8_gemm(XqT, api.E4M3, api.MAJOR_K, GqT, api.E5M2, api.MAJOR_K, dW1, si_x, si_g)
    torch.cuda.synchronize()
    assert torch.equal(dW0.view(torch.int32), dW1.view(torch.int32))


def test_full_size_activation_sampled():
    """activations of the hidden-4096 layer, [8192 x 4096] bf16: random 128 x 128 tiles and the four corner
    tiles of both outputs against the oracle, amax over the whole tensor"""
    T, I = 8192, 4096
    X = synth.activations(T * I, 3, device=DEV).view(T, I)
    out = torch.empty(T, I, dtype=torch.uint8, device=DEV)
    out_t = torch.empty(I, T, dtype=torch.uint8, device=DEV)
    amax = _scalar(-1.0)
    scale = 3.25
    api.fp8_quantize_transpose(X, api.E4M3, _scalar(scale), out, out_t, amax)
    torch.cuda.synchronize()
    xb = to_np_bits(X)
    assert amax.cpu().numpy().view(np.uint32)[0] == oracle.amax_bits(xb.reshape(-1), THREADS)
    rng = np.random.default_rng(0)
    tiles = [(0, 0), (0, I // 128 - 1), (T // 128 - 1, 0), (T // 128 - 1, I // 128 - 1)]
    tiles += [(int(a), int(b)) for a, b in zip(rng.integers(0, T // 128, 24), rng.integers(0, I // 128, 24))]
    out_h, out_t_h = out.cpu().numpy(), out_t.cpu().numpy()
    for tr, tc in tiles:
        blk = np.ascontiguousarray(xb[tr * 128:(tr + 1) * 128, tc * 128:(tc + 1) * 128])
        want = oracle.quantize(blk.reshape(-1), np.float32(scale), oracle.E4M3).reshape(128, 128)
        assert np.array_equal(out_h[tr * 128:(tr + 1) * 128, tc * 128:(tc + 1) * 128], want), (tr, tc)
        assert np.array_equal(out_t_h[tc * 128:(tc + 1) * 128, tr * 128:(tr + 1) * 128], want.T), (tr, tc)
    # every row-major code equals fp8_quantize's (itself checked against the oracle elsewhere), and the transposed
    # matrix is its transpose, everywhere
    ref = torch.empty(T * I, dtype=torch.uint8, device=DEV)
    api.fp8_quantize(X.view(-1), api.E4M3, _scalar(scale), ref)
    assert torch.equal(ref.view(T, I), out) and torch.equal(out.t(), out_t)
