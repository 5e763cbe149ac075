"""GPU parity of amax / scale / quantize / dequantize against the CPU oracle: bit-exact.
Everything goes through the C ABI (paper_2209_05433_b200.api)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2209_05433_b200 import api, synth
from tests._util import THREADS, same_with_nan, to_np_bits

pytestmark = pytest.mark.gpu

DEV = "cuda"
FMTS = [oracle.E4M3, oracle.E5M2]


def _scalar(v):
    return torch.tensor([v], dtype=torch.float32, device=DEV)


def _quantize_gpu(x, fmt, scale, overflow=api.SATURATE, with_amax=False):
    out = torch.full((x.numel() + 64,), 0xA5, dtype=torch.uint8, device=DEV)    # guard band behind the output
    view = out[: x.numel()]
    amax = _scalar(-1.0) if with_amax else None
    api.fp8_quantize(x, fmt, _scalar(scale), view, overflow, amax)
    torch.cuda.synchronize()
    assert bool((out[x.numel():] == 0xA5).all()), "wrote past the end of the output"
    return view.cpu().numpy(), (amax.cpu().numpy().view(np.uint32)[0] if with_amax else None)


def _assert_codes(got, want, x_np):
    bad = np.nonzero(got != want)[0]
    assert bad.size == 0, "%d mismatches, first: %s" % (
        bad.size, [(int(i), x_np[i], hex(got[i]), hex(want[i])) for i in bad[:6]])


def _all_bf16():
    bits = torch.arange(1 << 16, dtype=torch.int32).to(torch.int16)
    return bits.view(torch.bfloat16)


# -------------------------------------------------------------- quantize --

@pytest.mark.parametrize("fmt", FMTS)
@pytest.mark.parametrize("overflow", [api.SATURATE, api.NOSAT])
def test_quantize_every_bf16_value(fmt, overflow):
    x = _all_bf16().to(DEV)
    xb = to_np_bits(x)
    for scale in (1.0, 0.37, 121.08108, 2.0 ** -7, 3.0e4, 1e-30, 3.0e38):
        got, _ = _quantize_gpu(x, fmt, scale, overflow)
        want = oracle.quantize(xb, np.float32(scale), fmt, overflow)
        _assert_codes(got, want, xb)


@pytest.mark.parametrize("fmt", FMTS)
@pytest.mark.parametrize("overflow", [api.SATURATE, api.NOSAT])
def test_quantize_fp32_sweep(fmt, overflow):
    rng = np.random.default_rng(42 + fmt)
    t = oracle.decode_table(fmt)
    fin = t[np.isfinite(t)]
    mags = np.unique(np.abs(fin))
    mids = (mags[:-1] + mags[1:]) / 2
    pts = np.concatenate([mags, mids, [464.0, 480.0, 61440.0, 65536.0]]).astype(np.float32)
    b = pts.view(np.uint32).astype(np.int64)
    near = np.concatenate([np.clip(b + d, 0, 0x7F7FFFFF) for d in range(-3, 4)]).astype(np.uint32).view(np.float32)
    rand = rng.integers(0, 1 << 32, size=1 << 22, dtype=np.uint64).astype(np.uint32).view(np.float32)
    logu = (np.exp2(rng.uniform(-24, 18, size=1 << 21)) * rng.choice([-1.0, 1.0], size=1 << 21)).astype(np.float32)
    special = np.array([0.0, -0.0, np.inf, -np.inf, np.nan, 1e-45, -1e-45, 1e-39, 3.4e38, -3.4e38], dtype=np.float32)
    neg_nan = np.array([0xFFC00000, 0xFF800001, 0x7F800001], dtype=np.uint32).view(np.float32)
    x_np = np.concatenate([near, -near, rand, logu, special, neg_nan])
    x = torch.from_numpy(x_np).to(DEV)
    for scale in (1.0, 0.7310586):
        got, _ = _quantize_gpu(x, fmt, scale, overflow)
        want = oracle.quantize(x_np, np.float32(scale), fmt, overflow, threads=THREADS)
        _assert_codes(got, want, x_np)


@pytest.mark.parametrize("fmt", FMTS)
def test_quantize_scaled_overflow_to_infinity_is_special(fmt):
    # a finite input whose scaled value overflows binary32 becomes a special value, not the maximum
    x_np = np.array([3e38, -3e38, 1.0, 2e38] * 4, dtype=np.float32)
    got, _ = _quantize_gpu(torch.from_numpy(x_np).to(DEV), fmt, 4.0)
    want = oracle.quantize(x_np, np.float32(4.0), fmt)
    _assert_codes(got, want, x_np)
    assert want[0] == (0x7F if fmt == oracle.E4M3 else 0x7C)


@pytest.mark.parametrize("wide", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("n", [0, 1, 3, 7, 8, 9, 15, 16, 17, 31, 33, 1000, 4099, (1 << 20) - 1, (1 << 20) + 1])
def test_quantize_ragged_sizes_and_fused_amax(wide, n):
    x = synth.normal_laplace_mixture(n, 1, synth.T_ID, dtype=wide, device=DEV)
    x_np = to_np_bits(x)
    for fmt in FMTS:
        got, amax_bits = _quantize_gpu(x, fmt, 3.3, with_amax=True)
        want = oracle.quantize(x_np, np.float32(3.3), fmt, threads=THREADS)
        _assert_codes(got, want, x_np)
        assert amax_bits == oracle.amax_bits(x_np)


@pytest.mark.parametrize("wide", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("in_off,out_off", [(1, 0), (0, 1), (3, 5), (4, 4), (8, 8), (16, 3)])
def test_quantize_and_amax_unaligned_pointers(wide, in_off, out_off):
    n = 70001
    base = synth.normal_laplace_mixture(n + 64, 7, synth.T_ID, dtype=wide, device=DEV)
    x = base[in_off: in_off + n]
    x_np = to_np_bits(x)
    out = torch.full((n + 128,), 0x5A, dtype=torch.uint8, device=DEV)
    view = out[out_off: out_off + n]
    amax = _scalar(-1.0)
    api.fp8_quantize(x, oracle.E4M3, _scalar(2.5), view, api.SATURATE, amax)
    torch.cuda.synchronize()
    _assert_codes(view.cpu().numpy(), oracle.quantize(x_np, np.float32(2.5), oracle.E4M3), x_np)
    assert bool((out[:out_off] == 0x5A).all()) and bool((out[out_off + n:] == 0x5A).all())
    assert amax.cpu().numpy().view(np.uint32)[0] == oracle.amax_bits(x_np)
    a2 = _scalar(-1.0)
    api.fp8_amax(x, a2)
    assert a2.cpu().numpy().view(np.uint32)[0] == oracle.amax_bits(x_np)


# ------------------------------------------------------------------ amax --

@pytest.mark.parametrize("wide", [torch.float32, torch.bfloat16])
def test_amax_values_and_specials(wide):
    for n in (0, 1, 5, 8, 1023, 65536, (1 << 22) + 3):
        x = synth.activations(n, 3, dtype=wide, device=DEV)
        a = _scalar(-1.0)
        api.fp8_amax(x, a)
        assert a.cpu().numpy().view(np.uint32)[0] == oracle.amax_bits(to_np_bits(x)), n
    x = synth.activations(1 << 20, 3, dtype=wide, device=DEV)
    a = _scalar(0.0)
    x[12345] = float("-inf")
    api.fp8_amax(x, a)
    assert a.item() == float("inf")
    x[777777] = float("nan")
    api.fp8_amax(x, a)
    assert a.cpu().numpy().view(np.uint32)[0] == 0x7FC00000
    x[777777] = 1.0
    x[(1 << 20) - 1] = float("nan")         # in the last item
    api.fp8_amax(x, a)
    assert a.cpu().numpy().view(np.uint32)[0] == 0x7FC00000


@pytest.mark.parametrize("fmt", FMTS)
def test_scale_from_amax(fmt):
    rng = np.random.default_rng(8)
    vals = np.concatenate([np.exp2(rng.uniform(-140, 127, size=400)),
                           [0.0, np.inf, np.nan, 1.0, 448.0, 57344.0, 1e-44, 3.4e38]]).astype(np.float32)
    s, si = _scalar(0.0), _scalar(0.0)
    for v in vals:
        api.fp8_scale_from_amax(_scalar(float(v)), fmt, s, si)
        ws, wsi = oracle.scale_from_amax(v, fmt)
        assert s.cpu().numpy().view(np.uint32)[0] == np.array([ws]).view(np.uint32)[0], v
        assert si.cpu().numpy().view(np.uint32)[0] == np.array([wsi]).view(np.uint32)[0], v


# ------------------------------------------------------------ dequantize --

@pytest.mark.parametrize("fmt", FMTS)
@pytest.mark.parametrize("wide,name", [(torch.float32, "f32"), (torch.bfloat16, "bf16")])
def test_dequantize_every_code_and_ragged_sizes(fmt, wide, name):
    rng = np.random.default_rng(5)
    for n, si in ((256, 1.0), (256, 0.0082589), (256, 1e-38), (256, 3e35), (1, 0.5), (7, 0.5), (9, 0.5),
                  (4097, 0.25), ((1 << 20) + 5, 0.013)):
        codes_np = np.arange(256, dtype=np.uint8) if n == 256 else rng.integers(0, 256, size=n, dtype=np.uint16).astype(np.uint8)
        codes = torch.from_numpy(codes_np).to(DEV)
        out = torch.zeros(n + 16, dtype=wide, device=DEV)
        api.fp8_dequantize(codes, fmt, _scalar(si), out[:n])
        torch.cuda.synchronize()
        got = to_np_bits(out[:n])
        want = oracle.dequantize(codes_np, np.float32(si), fmt, name, threads=THREADS)
        ok = same_with_nan(got, want, name)
        assert ok.all(), (n, si, np.nonzero(~ok)[0][:5])
        assert bool((out[n:] == 0).all())


def test_dequantize_unaligned():
    n = 50001
    codes_np = np.random.default_rng(6).integers(0, 256, size=n + 32, dtype=np.uint16).astype(np.uint8)
    codes = torch.from_numpy(codes_np).to(DEV)
    for off_in, off_out in ((1, 0), (0, 1), (3, 2)):
        out = torch.zeros(n + 16, dtype=torch.bfloat16, device=DEV)
        api.fp8_dequantize(codes[off_in: off_in + n], oracle.E5M2, _scalar(0.5), out[off_out: off_out + n])
        got = to_np_bits(out[off_out: off_out + n])
        want = oracle.dequantize(codes_np[off_in: off_in + n], np.float32(0.5), oracle.E5M2, "bf16")
        assert same_with_nan(got, want, "bf16").all()


# ------------------------------------------- the workloads' cast steps --

def test_config1_casts():
    """tiny case: fp32 256x256 N(0,1) with 0.5% of entries x64; amax -> scale -> E4M3, in full"""
    for tid in (synth.A_ID, synth.B_ID):
        x = synth.normal_with_scaled_outliers(256 * 256, 0, tid, 0.005, 64.0, device=DEV)
        x_np = to_np_bits(x)
        a, s, si = _scalar(0.0), _scalar(0.0), _scalar(0.0)
        out = torch.empty(x.numel(), dtype=torch.uint8, device=DEV)
        api.fp8_amax(x, a)
        api.fp8_scale_from_amax(a, api.E4M3, s, si)
        api.fp8_quantize(x, api.E4M3, s, out)
        want_amax = oracle.amax(x_np)
        ws, wsi = oracle.scale_from_amax(want_amax, oracle.E4M3)
        assert a.item() == want_amax and s.item() == ws and si.item() == wsi
        _assert_codes(out.cpu().numpy(), oracle.quantize(x_np, ws, oracle.E4M3), x_np)
        assert out.cpu().numpy().view(np.uint8).max() >= 0x7E       # the maximum lands on the top code


@pytest.mark.parametrize("log2n", [20, 24])
def test_config2_small_sizes_in_full(log2n):
    n = 1 << log2n
    x = synth.normal_laplace_mixture(n, 1, synth.T_ID, device=DEV)
    x_np = to_np_bits(x)
    for fmt in FMTS:
        a, s, si = _scalar(0.0), _scalar(0.0), _scalar(0.0)
        codes = torch.empty(n, dtype=torch.uint8, device=DEV)
        back = torch.empty(n, dtype=torch.bfloat16, device=DEV)
        api.fp8_amax(x, a)
        api.fp8_scale_from_amax(a, fmt, s, si)
        api.fp8_quantize(x, fmt, s, codes)
        api.fp8_dequantize(codes, fmt, si, back)
        ws, wsi = oracle.scale_from_amax(oracle.amax(x_np, THREADS), fmt)
        assert s.item() == ws and si.item() == wsi
        wc = oracle.quantize(x_np, ws, fmt, threads=THREADS)
        _assert_codes(codes.cpu().numpy(), wc, x_np)
        wb = oracle.dequantize(wc, wsi, fmt, "bf16", threads=THREADS)
        assert same_with_nan(to_np_bits(back), wb, "bf16").all()


@pytest.mark.parametrize("log2n", [28, 30])
def test_config2_large_sizes_sampled(log2n):
    """full-size launch as the bench times it; the oracle checks the first and last 2^20 elements,
    32 random 64Ki blocks, and the exact amax of the whole tensor."""
    n = 1 << log2n
    x = synth.normal_laplace_mixture(n, 1, synth.T_ID, device=DEV)
    x_host = to_np_bits(x)
    rng = np.random.default_rng(log2n)
    blocks = [(0, 1 << 20), (n - (1 << 20), n)] + [(int(b) << 16, (int(b) + 1) << 16) for b in rng.integers(0, n >> 16, size=32)]
    for fmt in FMTS:
        a, s, si, a2 = _scalar(0.0), _scalar(0.0), _scalar(0.0), _scalar(0.0)
        codes = torch.empty(n, dtype=torch.uint8, device=DEV)
        back = torch.empty(n, dtype=torch.bfloat16, device=DEV)
        api.fp8_amax(x, a)
        api.fp8_scale_from_amax(a, fmt, s, si)
        api.fp8_quantize(x, fmt, s, codes, api.SATURATE, a2)
        api.fp8_dequantize(codes, fmt, si, back)
        torch.cuda.synchronize()
        want_amax_bits = oracle.amax_bits(x_host, THREADS)         # the whole tensor, on the host
        assert a.cpu().numpy().view(np.uint32)[0] == want_amax_bits == a2.cpu().numpy().view(np.uint32)[0]
        ws, wsi = oracle.scale_from_amax(np.array([want_amax_bits], dtype=np.uint32).view(np.float32)[0], fmt)
        assert s.item() == ws and si.item() == wsi
        for lo, hi in blocks:
            x_np = x_host[lo:hi]
            wc = oracle.quantize(x_np, ws, fmt, threads=THREADS)
            _assert_codes(codes[lo:hi].cpu().numpy(), wc, x_np)
            wb = oracle.dequantize(wc, wsi, fmt, "bf16", threads=THREADS)
            assert same_with_nan(to_np_bits(back[lo:hi]), wb, "bf16").all()
        del codes, back
    del x
    torch.cuda.empty_cache()


# ------------------------------------------ fused current scaling (one launch) --

@pytest.mark.parametrize("wide", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("n", [0, 1, 7, 8, 9, 1000, 4099, 1 << 20, (1 << 20) + 3, 1 << 22, (1 << 24) + 17])
def test_quantize_current_equals_three_calls_and_oracle(wide, n):
    x = synth.activations(n, 3, dtype=wide, device=DEV)
    x_np = to_np_bits(x)
    for fmt in FMTS:
        for overflow in (api.SATURATE, api.NOSAT):
            a, s, si = _scalar(-1.0), _scalar(-1.0), _scalar(-1.0)
            out = torch.full((n + 64,), 0xA5, dtype=torch.uint8, device=DEV)
            for _ in range(2):                                  # twice in a row: the workspace is left clean
                api.fp8_quantize_current(x, fmt, out[:n], a, s, si, overflow)
            torch.cuda.synchronize()
            assert api.fp8_async_status()[0] == 0
            want_amax_bits = oracle.amax_bits(x_np, THREADS)
            ws, wsi = oracle.scale_from_amax(np.array([want_amax_bits], dtype=np.uint32).view(np.float32)[0], fmt)
            assert a.cpu().numpy().view(np.uint32)[0] == want_amax_bits
            assert s.item() == ws and si.item() == wsi
            _assert_codes(out[:n].cpu().numpy(), oracle.quantize(x_np, ws, fmt, overflow, threads=THREADS), x_np)
            assert bool((out[n:] == 0xA5).all())
            assert bool((api.current_scaling_workspace(x.device) == 0).all())


@pytest.mark.parametrize("wide", [torch.float32, torch.bfloat16])
def test_quantize_current_at_the_shared_memory_capacity(wide):
    """the largest tensor the shared-memory-resident kernel takes (every SM's slice full), one item more (the general
    one-launch kernel), and the largest with a NaN in the last slice: same amax, scales and codes as the oracle"""
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    epi = 8 if wide == torch.bfloat16 else 4
    full = sms * 14336 * epi                                   # 224 KB of 16-byte items per SM
    for n, poke in ((full, None), (full + epi, None), (full, float("nan")), (full - 1024 * epi * 3, float("inf"))):
        x = synth.normal_laplace_mixture(n, 13, synth.T_ID, dtype=wide, device=DEV)
        if poke is not None:
            x[n - 5] = poke
        x_np = to_np_bits(x)
        a, s, si = _scalar(-1.0), _scalar(-1.0), _scalar(-1.0)
        out = torch.full((n + 64,), 0xA5, dtype=torch.uint8, device=DEV)
        api.fp8_quantize_current(x, api.E5M2, out[:n], a, s, si)
        torch.cuda.synchronize()
        assert api.fp8_async_status()[0] == 0
        want_bits = oracle.amax_bits(x_np, THREADS)
        ws, wsi = oracle.scale_from_amax(np.array([want_bits], dtype=np.uint32).view(np.float32)[0], oracle.E5M2)
        assert a.cpu().numpy().view(np.uint32)[0] == want_bits and s.item() == ws and si.item() == wsi
        _assert_codes(out[:n].cpu().numpy(), oracle.quantize(x_np, ws, oracle.E5M2, threads=THREADS), x_np)
        assert bool((out[n:] == 0xA5).all())
        assert bool((api.current_scaling_workspace(x.device) == 0).all())
        del x, out
    torch.cuda.empty_cache()


def test_quantize_current_specials_and_unaligned():
    n = 100003
    base = synth.normal_laplace_mixture(n + 16, 9, synth.T_ID, dtype=torch.bfloat16, device=DEV)
    for off, poke in ((0, float("nan")), (0, float("inf")), (3, None)):        # offset 3 takes the three-call path
        x = base[off: off + n].clone() if off == 0 else base[off: off + n]
        if poke is not None:
            x[n // 2] = poke
        x_np = to_np_bits(x)
        a, s, si = _scalar(-1.0), _scalar(-1.0), _scalar(-1.0)
        out = torch.empty(n, dtype=torch.uint8, device=DEV)
        api.fp8_quantize_current(x, api.E4M3, out, a, s, si)
        want_bits = oracle.amax_bits(x_np)
        ws, wsi = oracle.scale_from_amax(np.array([want_bits], dtype=np.uint32).view(np.float32)[0], oracle.E4M3)
        assert a.cpu().numpy().view(np.uint32)[0] == want_bits and s.item() == ws and si.item() == wsi
        _assert_codes(out.cpu().numpy(), oracle.quantize(x_np, ws, oracle.E4M3), x_np)


# ------------------------------- simulated FP8 round trip and power-of-two scale --

@pytest.mark.parametrize("fmt", FMTS)
def test_scale_pow2_from_amax(fmt):
    rng = np.random.default_rng(18)
    vals = np.concatenate([np.exp2(rng.uniform(-140, 127, size=300)), [0.0, np.inf, np.nan, 1.0, 448.0, 57344.0, 1e-44, 3.4e38]]).astype(np.float32)
    s, si = _scalar(0.0), _scalar(0.0)
    for v in vals:
        api.fp8_scale_pow2_from_amax(_scalar(float(v)), fmt, s, si)
        ws, wsi = oracle.scale_pow2_from_amax(v, fmt)
        assert s.cpu().numpy().view(np.uint32)[0] == np.array([ws]).view(np.uint32)[0], v
        assert si.cpu().numpy().view(np.uint32)[0] == np.array([wsi]).view(np.uint32)[0], v


@pytest.mark.parametrize("wide,name", [(torch.float32, "f32"), (torch.bfloat16, "bf16")])
@pytest.mark.parametrize("fmt", FMTS)
def test_fake_quantize_equals_quantize_then_dequantize(wide, name, fmt):
    for n, off in ((0, 0), (5, 0), (4099, 0), ((1 << 20) + 7, 0), (70001, 3)):
        base = synth.normal_laplace_mixture(n + 16, 11, synth.T_ID, dtype=wide, device=DEV)
        x = base[off: off + n]
        if n > 100:
            x = x.clone() if off == 0 else x
            x[7] = float("nan"); x[8] = float("-inf"); x[9] = 1e30
        x_np = to_np_bits(x)
        for overflow in (api.SATURATE, api.NOSAT):
            for scale, scale_inv in ((3.0, 1.0 / 3.0), (0.25, 4.0)):
                out = torch.zeros(n + 16, dtype=wide, device=DEV)
                api.fp8_fake_quantize(x, fmt, _scalar(scale), _scalar(scale_inv), out[off: off + n] if off else out[:n], overflow)
                torch.cuda.synchronize()
                got = to_np_bits(out[off: off + n] if off else out[:n])
                want = oracle.fake_quantize(x_np, np.float32(scale), np.float32(scale_inv), fmt, overflow, threads=THREADS)
                ok = same_with_nan(got, want, name)
                assert ok.all(), (n, off, overflow, scale, np.nonzero(~ok)[0][:5])


def test_fake_quantize_every_bf16_value():
    x = _all_bf16().to(DEV)
    xb = to_np_bits(x)
    for fmt in FMTS:
        out = torch.empty_like(x)
        api.fp8_fake_quantize(x, fmt, _scalar(0.37), _scalar(1.0 / 0.37), out)
        want = oracle.fake_quantize(xb, np.float32(0.37), np.float32(1.0 / 0.37), fmt)
        assert same_with_nan(to_np_bits(out), want, "bf16").all()
