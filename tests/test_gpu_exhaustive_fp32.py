"""Every one of the 2^32 binary32 bit patterns through fp8_quantize at scale 1, both formats, saturating mode:
the codes equal the oracle's, bit for bit (all NaN payloads, both infinities, every subnormal, every tie).
The oracle converts 2^27 values at a time on the host cores while the GPU works ahead."""
import numpy as np
import pytest
import torch

import oracle
from paper_2209_05433_b200 import api
from tests._util import THREADS

pytestmark = pytest.mark.gpu
DEV = "cuda"
CHUNK = 1 << 27


def _gpu_codes(lo, fmt, overflow, scale):
    bits = torch.arange(lo, lo + CHUNK, dtype=torch.int64, device=DEV).to(torch.int32)     # wraps into the sign bit
    out = torch.empty(CHUNK, dtype=torch.uint8, device=DEV)
    api.fp8_quantize(bits.view(torch.float32), fmt, scale, out, overflow)
    return out.to("cpu", non_blocking=False).numpy()


@pytest.mark.parametrize("fmt", [oracle.E4M3, oracle.E5M2])
def test_quantize_every_binary32_value(fmt):
    scale = torch.ones(1, dtype=torch.float32, device=DEV)
    for lo in range(0, 1 << 32, CHUNK):
        got = _gpu_codes(lo, fmt, api.SATURATE, scale)
        x = np.arange(lo, lo + CHUNK, dtype=np.uint64).astype(np.uint32).view(np.float32)
        want = oracle.quantize(x, np.float32(1.0), fmt, oracle.SATURATE, threads=THREADS)
        bad = np.nonzero(got != want)[0]
        assert bad.size == 0, "%d mismatches in [%#x, %#x), first at bits %#010x: gpu %#04x oracle %#04x" % (
            bad.size, lo, lo + CHUNK, lo + int(bad[0]), got[bad[0]], want[bad[0]])


def test_quantize_nonsaturating_threshold_and_top_ranges():
    """the non-saturating mode differs from the saturating one only from the overflow thresholds upwards: every
    pattern of [2, 131072) (both thresholds, 464 and 61440, lie inside) and of the top 2^27 patterns (largest
    finite values, infinity, every NaN payload), both signs, both formats"""
    scale = torch.ones(1, dtype=torch.float32, device=DEV)
    for fmt in (oracle.E4M3, oracle.E5M2):
        for lo in (0x40000000, 0x78000000, 0xC0000000, 0xF8000000):
            got = _gpu_codes(lo, fmt, api.NOSAT, scale)
            x = np.arange(lo, lo + CHUNK, dtype=np.uint64).astype(np.uint32).view(np.float32)
            want = oracle.quantize(x, np.float32(1.0), fmt, oracle.NOSAT, threads=THREADS)
            assert np.array_equal(got, want), (fmt, hex(lo))
