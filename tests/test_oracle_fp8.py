"""Pins for the e4m3 decode of the FP8-cache oracle: torch's float8_e4m3fn conversion on all 256
codes (a library routine the oracle does not use), the format's landmarks, and bf16 rounding against
torch's."""
import numpy as np
import torch

from oracle import fp8


def test_decode_matches_torch_on_every_code():
    codes = np.arange(256, dtype=np.uint8)
    ref = torch.from_numpy(codes).view(torch.float8_e4m3fn).to(torch.float64).numpy()
    got = fp8.decode_e4m3(codes)
    assert np.array_equal(np.isnan(got), np.isnan(ref))
    ok = ~np.isnan(ref)
    assert np.array_equal(got[ok], ref[ok])


def test_format_landmarks():
    d = fp8.decode_e4m3
    assert d([0x00])[0] == 0.0 and d([0x80])[0] == 0.0 and np.signbit(d([0x80])[0])
    assert d([0x38])[0] == 1.0 and d([0xB8])[0] == -1.0          # exponent field 7 = bias
    assert d([0x7E])[0] == 448.0                                 # largest finite value
    assert d([0x01])[0] == 2.0 ** -9 and d([0x08])[0] == 2.0 ** -6   # smallest subnormal / normal
    assert np.isnan(d([0x7F])[0]) and np.isnan(d([0xFF])[0])


def test_bf16_rounding_matches_torch():
    rng = np.random.default_rng(0)
    x = np.concatenate([rng.standard_normal(5000).astype(np.float32) * 37.0,
                        np.array([1.00390625, 1.01171875, 3.0e38, -2.5e-40, 0.0], np.float32)])  # ties, extremes
    ref = torch.from_numpy(x).to(torch.bfloat16).to(torch.float32).numpy()
    assert np.array_equal(fp8.bf16_round(x), ref)


def test_dequant_applies_the_scale_per_sequence_and_head():
    codes = np.full((2, 3, 2, 4), 0x38, np.uint8)               # all ones
    scale = np.array([[0.5, 2.0], [3.0, 1.0 / 3.0]], np.float32)
    out = fp8.dequant_cache(codes, scale)
    assert out.shape == codes.shape
    for s in range(2):
        for h in range(2):
            want = torch.tensor(scale[s, h]).to(torch.bfloat16).float().item()
            assert (out[s, :, h, :] == want).all()
    assert (fp8.dequant_cache(codes) == 1.0).all()
