"""Pins for the oracle's 16-bit sketch quantisation: its rounding against numpy's float16 and torch's
bfloat16 conversions (library routines, round to nearest even), saturation, and the fp32 merge."""
import numpy as np
import torch

from oracle import FMT_BF16, FMT_F16, merge16, quantize16


def samples():
    rng = np.random.default_rng(0)
    x = np.concatenate([
        rng.standard_normal(20000).astype(np.float32) * np.float32(10.0) ** rng.integers(-9, 5, 20000).astype(np.float32),
        np.array([0.0, -0.0, 1.0, -1.0, 65504.0, 65519.9, -65519.9, 6.1035156e-05, 5.9604645e-08, 2.9802322e-08,
                  2.9802326e-08, 1e-10, 2049.0, 2051.0, 1.00048828125, 1.0009765625 + 2**-12], np.float32),
        (np.arange(0, 70000, 7)).astype(np.float32) * np.float32(2**-24),      # the binary16 subnormal range
    ])
    return x.astype(np.float32)


def test_binary16_rounding_matches_numpy():
    x = samples()
    x = x[np.abs(x) < 65520]                      # beyond that numpy gives inf; the oracle saturates (next test)
    got = quantize16(x, FMT_F16)
    want = x.astype(np.float16).view(np.uint16)
    assert (got == want).all()


def test_binary16_saturates():
    x = np.array([65520.0, 1e6, -70000.0, 3e38], np.float32)
    assert quantize16(x, FMT_F16).tolist() == [0x7BFF, 0x7BFF, 0xFBFF, 0x7BFF]


def test_bfloat16_rounding_matches_torch():
    x = samples()
    got = quantize16(x, FMT_BF16)
    want = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert (got == want).all()


def test_merge16_decodes_and_sums_in_worker_order():
    rng = np.random.default_rng(1)
    W, n = 5, 3000
    x = rng.standard_normal((W, n)).astype(np.float32) * 100
    for fmt, dec in ((FMT_F16, lambda q: q.view(np.float16).astype(np.float32)),
                     (FMT_BF16, lambda q: torch.from_numpy(q.view(np.int16)).view(torch.bfloat16).float().numpy())):
        q = quantize16(x, fmt)
        want = np.zeros(n, np.float32)
        for w in range(W):
            want = want + dec(q[w])
        assert (merge16(q, fmt) == want).all()
        # quantisation error of one value: half a unit in the last place of the 16-bit format
        rel = 2.0 ** -11 if fmt == FMT_F16 else 2.0 ** -8
        assert (np.abs(dec(q) - x) <= rel * np.abs(x) + 1e-7).all()
